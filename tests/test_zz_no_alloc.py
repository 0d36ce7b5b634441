"""corun_gemm_static: the GEMM for callers that cannot allocate device memory
(arena-managed processes, loops that cannot take an allocation's device-wide
synchronisation).  It must give what the allocating entry point gives, on
repeated calls that share the library's one scratch array.  Collected last on
purpose: a failure here stops nothing else."""
import numpy as np
import pytest

from paper_2608_14376_b200 import synth

pytestmark = pytest.mark.gpu


def _inputs(torch, R, N, K, seed, with_host=False):
    rng = np.random.default_rng(seed)
    Wb = synth.f32_to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    X = rng.standard_normal((R, K)).astype(np.float32)
    Wt = torch.from_numpy(Wb.view(np.int16).copy()).view(torch.bfloat16).cuda()
    if with_host:
        return Wt, torch.from_numpy(X).cuda(), Wb, X
    return Wt, torch.from_numpy(X).cuda()


def test_static_scratch_gemm_equals_allocating_gemm_on_two_calls_in_a_row(orc):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    # two different problems back to back: the second call finds the first one's leftovers in the scratch
    cases = [(16, 4096, 4096, 1), (5, 1536, 256, 2)]
    for R, N, K, seed in cases:
        Wt, Xt, Wb, X = _inputs(torch, R, N, K, seed, with_host=True)
        got = corun.gemm_static(Wt, Xt).cpu().numpy()
        want = corun.debug_gemm(Wt, Xt).cpu().numpy()
        tol = 2e-5 * 0.02 * np.sqrt(K) * 4 + 1e-6          # the tolerance of the GEMM parity tests
        assert np.abs(got - want).max() <= tol
        assert np.abs(want).max() > 0.1
        # and against the oracle's definition of the product, as for the allocating entry point
        assert np.abs(got - orc.matmul_bf16(Wb, X)).max() <= tol
    # and the same problem twice gives the same bytes
    Wt, Xt = _inputs(torch, 9, 2048, 1024, 3)
    a = corun.gemm_static(Wt, Xt).cpu().numpy()
    b = corun.gemm_static(Wt, Xt).cpu().numpy()
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(a, corun.debug_gemm(Wt, Xt).cpu().numpy())


def test_sizes_beyond_the_scratch_are_refused():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    for R, N, K in [(17, 256, 256), (4, 8192 + 128, 256), (4, 256, 4096 + 64)]:
        Wt, Xt = _inputs(torch, R, N, K, 4)
        with pytest.raises(corun.CorunError) as ei:
            corun.gemm_static(Wt, Xt)
        assert ei.value.status == corun.ELIMIT
