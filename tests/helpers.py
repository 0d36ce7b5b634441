"""Shared helpers of the GPU tests."""
import numpy as np

from paper_2608_14376_b200 import synth


def have_gpu() -> bool:
    try:
        import torch

        return torch.cuda.is_available()
    except Exception:
        return False


def oracle_model(orc, sh, w_np):
    return orc.Model(orc.Shape(**sh.dict()), w_np)


def top2_gap(logits: np.ndarray) -> float:
    part = np.partition(logits, -2)[-2:]
    return float(part[1] - part[0])


class Tiny:
    """Tiny config of the baseline: weights on both sides + an oracle model."""

    def __init__(self, orc, seed=0):
        self.sh = synth.TINY
        self.w_np = synth.make_weights_numpy(self.sh, seed=seed)
        self.w_t = synth.weights_numpy_to_torch(self.w_np, "cuda")
        self.oracle = oracle_model(orc, self.sh, self.w_np)
