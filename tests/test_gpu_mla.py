"""Absorbed multi-head latent attention against its oracle, and row independence."""
import math

import numpy as np
import pytest

from oracle import mla_oracle as ml

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("nh,dc,dr,pairs", [(16, 512, 64, True), (4, 64, 8, True), (8, 128, 32, True), (16, 512, 24, True),
                                            (4, 64, 16, True), (16, 512, 64, False), (8, 128, 32, False), (4, 64, 16, False)])
def test_mla_attend_matches_oracle_and_rows_are_independent(nh, dc, dr, pairs):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    rng = np.random.default_rng(nh + dc)
    ctxs = [0, 1, 127, 128, 129, 700, 385]
    B, T = len(ctxs), 768
    q_lat = rng.standard_normal((B, nh, dc)).astype(np.float32)
    q_rope = rng.standard_normal((B, nh, dr)).astype(np.float32)
    cache = (rng.standard_normal((B, T, dc + dr)) * 0.5).astype(np.float16)
    scale = 1.0 / math.sqrt(dc + dr)
    dev = lambda a: torch.tensor(a).cuda().contiguous()
    out = corun.mla_attend(dev(q_lat), dev(q_rope), dev(cache), dev(np.array(ctxs, np.int32)), scale, pairs)
    torch.cuda.synchronize()
    out = out.cpu().numpy()
    eye = np.stack([np.eye(dc)] * nh)               # W_uk = W_uv = identity: the absorbed level itself
    worst = 0.0
    for b, n in enumerate(ctxs):
        if n == 0:
            assert not out[b].any()                  # a padding row is left alone
            continue
        C = cache[b, :n, :dc].astype(np.float64)
        Rk = cache[b, :n, dc:].astype(np.float64)
        ref = ml.attend_absorbed(q_lat[b], q_rope[b], C, Rk, eye, eye)
        worst = max(worst, float(np.abs(out[b] - ref).max()))
    # hi + lo pairs: fp32 accumulation chains of <= 576 and <= 512 terms on O(1) values.  Single fp16 operands:
    # queries rounded to 2^-11 relative move a score by <= 2^-11 * scale * sum |q_d c_d| (~ 1e-3 here: 576 terms of
    # ~0.4 times 0.04), which moves the weights, and so the outputs of size <= ~2, by that fraction at most;
    # the rounding of the weights themselves adds 2^-11 relative.
    assert worst <= (2e-5 if pairs else 4e-3), worst
    # the same rows in another order among other rows: byte-identical
    perm = [5, 2, 6]
    q2 = rng.standard_normal((B, nh, dc)).astype(np.float32); r2 = rng.standard_normal((B, nh, dr)).astype(np.float32)
    c2 = (rng.standard_normal((B, T, dc + dr)) * 0.5).astype(np.float16)
    ctx2 = np.array([300, 5, 64, 9, 0, 17, 640], np.int32)
    for i, src in enumerate(perm):
        q2[i], r2[i], c2[i], ctx2[i] = q_lat[src], q_rope[src], cache[src], ctxs[src]
    out2 = corun.mla_attend(dev(q2), dev(r2), dev(c2), dev(ctx2), scale, pairs).cpu().numpy()
    for i, src in enumerate(perm):
        assert out2[i].tobytes() == out[src].tobytes()


def test_mla_single_operands_need_the_tensor_path():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    z = lambda *s: torch.zeros(s, device="cuda")
    with pytest.raises(Exception):                   # d_rope = 8: only the FMA kernel takes it, and only with pairs
        corun.mla_attend(z(1, 4, 64), z(1, 4, 8), z(1, 128, 72).half(), torch.ones(1, dtype=torch.int32, device="cuda"), 1.0, False)


def _mla_case(nh, dc, dr, ctxs, T, seed):
    rng = np.random.default_rng(seed)
    B = len(ctxs)
    q_lat = rng.standard_normal((B, nh, dc)).astype(np.float32)
    q_rope = rng.standard_normal((B, nh, dr)).astype(np.float32)
    cache = (rng.standard_normal((B, T, dc + dr)) * 0.5).astype(np.float16)
    return q_lat, q_rope, cache


def _mla_worst(out, q_lat, q_rope, cache, ctxs, dc):
    nh = q_lat.shape[1]
    eye = np.stack([np.eye(dc)] * nh)
    worst = 0.0
    for b, n in enumerate(ctxs):
        C = cache[b, :n, :dc].astype(np.float64)
        Rk = cache[b, :n, dc:].astype(np.float64)
        ref = ml.attend_absorbed(q_lat[b], q_rope[b], C, Rk, eye, eye)
        worst = max(worst, float(np.abs(out[b] - ref).max()))
    return worst


@pytest.mark.parametrize("path", ["", "CORUN_MLA_UNPIPELINED", "CORUN_MLA_FMA"])
def test_mla_every_kernel_and_more_pieces_than_the_combine_fast_path(path):
    """The three kernels (selected by environment variable) on contexts around the chunk boundary and on one with
    more pieces than the combine kernel keeps in registers (18 chunks of 512, 71 splits of 128)."""
    import os

    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    nh, dc, dr = 4, 64, 16
    ctxs = [9000, 512, 513, 1024, 63]
    q_lat, q_rope, cache = _mla_case(nh, dc, dr, ctxs, 9216, seed=7)
    scale = 1.0 / math.sqrt(dc + dr)
    dev = lambda a: torch.tensor(a).cuda().contiguous()
    if path:
        os.environ[path] = "1"
    try:
        out = corun.mla_attend(dev(q_lat), dev(q_rope), dev(cache), dev(np.array(ctxs, np.int32)), scale)
        torch.cuda.synchronize()
        again = corun.mla_attend(dev(q_lat), dev(q_rope), dev(cache), dev(np.array(ctxs, np.int32)), scale)
        torch.cuda.synchronize()
    finally:
        if path:
            os.environ.pop(path, None)
    assert out.cpu().numpy().tobytes() == again.cpu().numpy().tobytes()
    assert _mla_worst(out.cpu().numpy(), q_lat, q_rope, cache, ctxs, dc) <= 2e-5


def test_mla_v2_widths_match_the_runtime_width_kernel_on_the_oracle():
    """d_c = 512, d_r = 64 takes the kernel with the widths compiled in: long contexts, several chunks."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    nh, dc, dr = 16, 512, 64
    ctxs = [2049, 1536, 511]
    q_lat, q_rope, cache = _mla_case(nh, dc, dr, ctxs, 2176, seed=11)
    scale = 1.0 / math.sqrt(dc + dr)                 # the oracle's scale for identity up-projections (d_nope = d_c)
    dev = lambda a: torch.tensor(a).cuda().contiguous()
    for pairs, tol in ((True, 2e-5), (False, 4e-3)):
        out = corun.mla_attend(dev(q_lat), dev(q_rope), dev(cache), dev(np.array(ctxs, np.int32)), scale, pairs)
        torch.cuda.synchronize()
        assert _mla_worst(out.cpu().numpy(), q_lat, q_rope, cache, ctxs, dc) <= tol


def test_mla_context_beyond_the_cache_is_cut():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    nh, dc, dr, T = 8, 128, 32, 640
    q_lat, q_rope, cache = _mla_case(nh, dc, dr, [T, T], T, seed=3)
    scale = 1.0 / math.sqrt(dc + dr)
    dev = lambda a: torch.tensor(a).cuda().contiguous()
    full = corun.mla_attend(dev(q_lat), dev(q_rope), dev(cache), dev(np.array([T, T], np.int32)), scale)
    over = corun.mla_attend(dev(q_lat), dev(q_rope), dev(cache), dev(np.array([T + 100, 1 << 30], np.int32)), scale)
    torch.cuda.synchronize()
    assert over.cpu().numpy().tobytes() == full.cpu().numpy().tobytes()
