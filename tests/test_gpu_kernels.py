"""GPU parity of single kernels against the oracle, through the C ABI."""
import numpy as np
import pytest

from paper_2608_14376_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch_cuda():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch


def _gemm_case(orc, torch, R, N, K, seed):
    from paper_2608_14376_b200 import corun

    rng = np.random.default_rng(seed)
    Wb = synth.f32_to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    X = rng.standard_normal((R, K)).astype(np.float32)
    Wt = torch.from_numpy(Wb.view(np.int16).copy()).view(torch.bfloat16).cuda()
    Xt = torch.from_numpy(X).cuda()
    out = corun.debug_gemm(Wt, Xt).cpu().numpy()
    ref = orc.matmul_bf16(Wb, X)
    return out, ref, Wt, Xt


# rows x weight rows x K: single tile, ragged N, several tiles, more k-blocks than CTAs, all 256 rows; 65..128 rows
# (two stacked blocks of 64 rows, the second one ragged or full), 129..256 rows (two row blocks of 128)
@pytest.mark.parametrize("R,N,K", [(8, 128, 64), (8, 512, 256), (5, 384, 768), (1, 2048, 256), (40, 200, 128),
                                   (64, 1536, 256), (64, 4096, 4096), (130, 1024, 1024), (256, 512, 512),
                                   (72, 640, 512), (100, 1024, 1024), (128, 4096, 2048), (200, 768, 1024)])
def test_gemm_matches_oracle(orc, torch_cuda, R, N, K):
    out, ref, _, _ = _gemm_case(orc, torch_cuda, R, N, K, seed=R + N + K)
    # split activations carry 16 significand bits: error << 1e-4 of the output scale (0.02 * sqrt(K))
    tol = 2e-5 * 0.02 * np.sqrt(K) * 4 + 1e-6
    assert np.abs(out - ref).max() <= tol, (np.abs(out - ref).max(), tol)


def test_gemm_rows_are_position_invariant(orc, torch_cuda):
    from paper_2608_14376_b200 import corun

    torch = torch_cuda
    out, _, Wt, Xt = _gemm_case(orc, torch, 64, 1024, 4096, seed=3)
    perm = torch.randperm(64, generator=torch.Generator().manual_seed(1)).cuda()
    out_p = corun.debug_gemm(Wt, Xt[perm].contiguous()).cpu().numpy()
    np.testing.assert_array_equal(out_p, out[perm.cpu().numpy()])
    # other rows' values cannot leak into a row
    Y = Xt.clone()
    Y[1:] = 1e30
    out_y = corun.debug_gemm(Wt, Y).cpu().numpy()
    np.testing.assert_array_equal(out_y[0], out[0])
    # repeated runs
    np.testing.assert_array_equal(corun.debug_gemm(Wt, Xt).cpu().numpy(), out)


@pytest.mark.parametrize("R", [100, 128, 200])
def test_gemm_rows_are_position_invariant_across_row_blocks(orc, torch_cuda, R):
    """Above 64 rows the rows sit in two blocks with an accumulator each: a row's bytes do not depend on the block
    it is in, nor on what the other block holds."""
    from paper_2608_14376_b200 import corun

    torch = torch_cuda
    out, _, Wt, Xt = _gemm_case(orc, torch, R, 1024, 2048, seed=5 + R)
    perm = torch.randperm(R, generator=torch.Generator().manual_seed(2)).cuda()
    out_p = corun.debug_gemm(Wt, Xt[perm].contiguous()).cpu().numpy()
    np.testing.assert_array_equal(out_p, out[perm.cpu().numpy()])
    Y = Xt.clone()
    Y[1:] = 1e30
    np.testing.assert_array_equal(corun.debug_gemm(Wt, Y).cpu().numpy()[0], out[0])
    # the same rows alone in a smaller matrix of the same row path (R rows -> the first 70 rows of an R-row call)
    Z = torch.zeros_like(Xt)
    Z[:70] = Xt[R - 70:]
    np.testing.assert_array_equal(corun.debug_gemm(Wt, Z).cpu().numpy()[:70], out[R - 70:])


def test_variate_matches_oracle(orc, torch_cuda):
    from paper_2608_14376_b200 import corun

    rng = np.random.default_rng(0)
    pairs = [(0, 0), (1042, 7), (2**63 + 11, 2**33 + 5)] + [
        (int(rng.integers(0, 2**63)), int(rng.integers(0, 4096))) for _ in range(1500)]
    for seed, t in pairs:
        assert corun.debug_variate(seed, t) == orc.variate_u24(seed, t)


def _check_sampler(orc, logits, T, top_p, us):
    from paper_2608_14376_b200 import corun

    rows = np.repeat(logits[None], len(us), axis=0)
    got = corun.debug_sample(rows, T, top_p, np.array(us, np.uint32))
    n_checked = 0
    # the plain fp64 definition of S decides the same token wherever its own margin exceeds the accuracy of
    # the specification's integer weights (2e-7 relative): checked on the GPU's tokens too
    plain, plain_margin = orc.sample_plain_many(logits, T, top_p, np.array(us, np.uint32))
    for k, (u, g) in enumerate(zip(us, got)):
        # the sampling weights are integers in a stated fp32 arithmetic: the decision is exact
        want, margin = orc.sample(logits, T, top_p, int(u))
        assert g == want, (u, g, want, margin)
        if plain_margin[k] >= 1e-6:
            assert g == plain[k], (u, g, int(plain[k]), float(plain_margin[k]))
        n_checked += 1
    return n_checked


@pytest.mark.parametrize("V", [2048, 151936])
def test_sampler_matches_oracle(orc, torch_cuda, V):
    rng = np.random.default_rng(V)
    us = [0, 1, (1 << 24) - 1, 1 << 23] + [int(x) for x in rng.integers(0, 1 << 24, 28)]
    logits = (rng.standard_normal(V) * 1.28).astype(np.float32)
    n = 0
    for T, top_p in [(0.7, 0.95), (1.0, 1.0), (0.6, 0.5), (0.7, 1e-6), (2.0, 0.999)]:
        n += _check_sampler(orc, logits, T, top_p, us)
    assert n == 5 * len(us)
    # greedy
    from paper_2608_14376_b200 import corun

    assert corun.debug_sample(logits, 0.0, 1.0, [5])[0] == int(np.argmax(logits))


def test_sampler_ties_and_degenerate_rows(orc, torch_cuda):
    from paper_2608_14376_b200 import corun

    rng = np.random.default_rng(5)
    us = [int(x) for x in rng.integers(0, 1 << 24, 32)]
    # heavily tied logits (quantised to 1/4): the nucleus edge falls inside a tie group
    tied = (np.round(rng.standard_normal(4096) * 4) / 4).astype(np.float32)
    assert _check_sampler(orc, tied, 0.7, 0.9, us) > 20
    assert _check_sampler(orc, tied, 1.0, 0.3, us) > 20
    # all equal
    flat = np.zeros(1000, np.float32)
    assert _check_sampler(orc, flat, 1.0, 0.5, us) > 20
    # more equal, or nearly equal, logits at the nucleus edge than the kernel keeps in shared memory
    assert _check_sampler(orc, np.zeros(8192, np.float32), 1.0, 0.5, us) > 20
    dense = (1.0 + rng.integers(0, 50, 6000) * 1.2e-7).astype(np.float32)
    assert _check_sampler(orc, dense, 0.7, 0.6, us) > 20
    mixed = np.concatenate([dense, (rng.standard_normal(3000) * 1.28).astype(np.float32)])
    assert _check_sampler(orc, mixed, 0.7, 0.9, us) > 20
    # one dominant token, very wide range
    wide = (rng.standard_normal(3000) * 30).astype(np.float32)
    assert _check_sampler(orc, wide, 0.7, 0.95, us) > 20
    # argmax picks the lowest id among equal maxima
    two = np.zeros(777, np.float32); two[[5, 300]] = 3.0
    assert corun.debug_sample(two, 0.0, 1.0, [0])[0] == 5


def test_a_bounded_wait_runs_out_and_the_context_stays_usable(orc, torch_cuda):
    """A one-CTA kernel waits, with the library's own wait routine and a limit of 1 ms, on a barrier nothing
    arrives at: the wait gives up, the kernel returns normally with its status word set and the call reports
    ETIMEOUT.  Nothing traps or faults, so an ordinary kernel launched afterwards works."""
    import ctypes as C
    import time

    import torch
    from paper_2608_14376_b200 import corun

    L = corun.lib()
    L.corun_debug_wait_probe.argtypes = [C.c_uint64, C.c_void_p]
    t0 = time.perf_counter()
    assert L.corun_debug_wait_probe(1_000_000, None) == corun.ETIMEOUT
    assert time.perf_counter() - t0 < 2.0
    assert L.corun_debug_wait_probe(10, None) == corun.EINVAL          # limits outside 1 us .. 100 ms are refused
    assert L.corun_debug_wait_probe(10**10, None) == corun.EINVAL
    # the device is fine: a GEMM against the oracle
    rng = np.random.default_rng(1)
    Wb = synth.f32_to_bf16_bits(rng.standard_normal((512, 256)).astype(np.float32) * 0.02)
    X = rng.standard_normal((3, 256)).astype(np.float32)
    Wt = torch.from_numpy(Wb.view(np.int16).copy()).view(torch.bfloat16).cuda()
    got = corun.debug_gemm(Wt, torch.from_numpy(X).cuda()).cpu().numpy()
    assert np.abs(got - orc.matmul_bf16(Wb, X)).max() < 1e-4
