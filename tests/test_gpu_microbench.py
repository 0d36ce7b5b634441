"""The micro-benchmark's kernels compute what they say (against numpy, both tilings), and the fixed tiling gives a
row the same bytes whatever the batch size is."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _torch():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch


@pytest.mark.parametrize("kind", [0, 1, 2])
def test_microbench_kernels_against_numpy_and_fixed_tiling_is_batch_invariant(kind):
    torch = _torch()
    from paper_2608_14376_b200 import corun

    N = 4096
    g = torch.Generator(device="cuda").manual_seed(kind)
    big = torch.randn((96, N), generator=g, device="cuda")
    xs = big.cpu().numpy().astype(np.float64)
    for variant in (0, 1):
        for R in (1, 5, 96):
            y, us, til = corun.microbench(kind, variant, big[:R].contiguous(), reps=2)
            x = xs[:R]
            if kind == 0:
                ref = x / np.sqrt((x * x).mean(axis=1, keepdims=True) + 1e-6)
            elif kind == 1:
                e = np.exp(x - x.max(axis=1, keepdims=True)); ref = e / e.sum(axis=1, keepdims=True)
            else:
                ref = x.sum(axis=0)
            assert us > 0 and til >= 1
            assert np.abs(y.cpu().numpy() - ref).max() <= 2e-5 * max(1.0, np.abs(ref).max())
    if kind < 2:      # a row's bytes under the fixed tiling do not depend on how many rows share the launch
        alone = corun.microbench(kind, 0, big[:1].contiguous(), reps=1)[0].cpu().numpy()
        among = corun.microbench(kind, 0, big, reps=1)[0].cpu().numpy()
        assert alone[0].tobytes() == among[0].tobytes()
