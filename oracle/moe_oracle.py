"""Plain CPU oracle of one Mixture-of-Experts feed-forward block at decode time.

TEST INFRASTRUCTURE ONLY: imported by ``tests/`` and by ``bench``-style cases that time the CPU
baseline.  It shares no code with the CUDA path and never imports it.

What it computes (the paper evaluates Mixture-of-Experts models -- Evaluation, "Setup" -- and notes,
in its comparison with LLM-42, that a small router perturbation changes the selected experts; it gives
no formulas, so the block is the standard one of the DeepSeek-V2-Lite shape the workload names):

    logits_e = <x, Wr[e]>                                   e = 0..E-1            (router)
    p        = softmax(logits)                              over all E experts
    S        = the top_k experts by p, ties to the lower expert id
    y        = sum_{e in S} p_e * FFN_e(x)  +  sum_s FFN_shared_s(x)              (no renormalisation of p)
    FFN(x)   = Wd @ (silu(Wg @ x) * (Wu @ x)),   silu(a) = a / (1 + exp(-a))

Readings (the paper is silent): gating is softmax-then-top-k; the selected probabilities are used as
they are (they sum to less than 1; the DeepSeek-V2-Lite convention) or, with ``renormalize``, divided by
their sum in descending-probability order (the Qwen3-MoE convention; the paper evaluates both families);
shared experts are always on with weight 1; the sum over the
selected experts runs in ascending expert id, the shared experts last.  Everything is fp64 on the
given (already bf16-valued) weights and fp32-valued inputs; loops are plain, one row and one expert
at a time.

Pins (tests/test_moe_oracle.py): a hand-computed routing example, the tie rule, top_k = E with identical
experts (= the dense FFN, because the probabilities sum to 1), one expert = the dense FFN written with
library matmuls, a brute-force scalar-loop restatement on a tiny case, row-permutation equivariance.
"""
from __future__ import annotations

import numpy as np


def silu(a: np.ndarray) -> np.ndarray:
    a = np.asarray(a, dtype=np.float64)
    return a / (1.0 + np.exp(-a))


def ffn(x: np.ndarray, Wg: np.ndarray, Wu: np.ndarray, Wd: np.ndarray) -> np.ndarray:
    """One expert on one row x [H]: Wg, Wu [F, H], Wd [H, F]."""
    x = np.asarray(x, dtype=np.float64)
    g = np.asarray(Wg, dtype=np.float64) @ x
    u = np.asarray(Wu, dtype=np.float64) @ x
    return np.asarray(Wd, dtype=np.float64) @ (silu(g) * u)


def router(x: np.ndarray, Wr: np.ndarray, top_k: int):
    """Row x [H], router weights Wr [E, H] -> (expert ids [top_k] by descending probability, ties to the
    lower id; their probabilities [top_k]; all probabilities [E])."""
    logits = np.asarray(Wr, dtype=np.float64) @ np.asarray(x, dtype=np.float64)
    z = np.exp(logits - logits.max())
    p = z / z.sum()
    order = sorted(range(len(p)), key=lambda e: (-p[e], e))
    ids = np.array(order[:top_k], dtype=np.int64)
    return ids, p[ids], p


def moe_ffn(X, Wr, Wg, Wu, Wd, shared, top_k: int, experts=None, renormalize: bool = False):
    """X [B, H]; Wr [E, H]; Wg, Wu [E, F, H]; Wd [E, H, F]; shared = list of (Wg, Wu, Wd) always-on
    experts.  ``experts`` ([B, top_k] ids) overrides the router's choice (their probabilities are still
    the router's), for comparing outputs when a near-tie was decided the other way in another precision.
    Returns (Y [B, H] fp64, ids [B, top_k], probs [B, top_k])."""
    X = np.asarray(X)
    B = X.shape[0]
    Y = np.zeros((B, X.shape[1]), dtype=np.float64)
    ids_out = np.zeros((B, top_k), dtype=np.int64)
    p_out = np.zeros((B, top_k), dtype=np.float64)
    for b in range(B):
        ids, ps, p_all = router(X[b], Wr, top_k)
        if experts is not None:
            ids = np.asarray(experts[b], dtype=np.int64)
            ps = p_all[ids]
        if renormalize:
            tot = 0.0
            for v in ps:                                      # in the order of ids: descending probability
                tot += v
            ps = ps / tot
        ids_out[b], p_out[b] = ids, ps
        weight = {int(e): float(w) for e, w in zip(ids, ps)}
        y = np.zeros(X.shape[1], dtype=np.float64)
        for e in sorted(weight):                              # ascending expert id
            y += weight[e] * ffn(X[b], Wg[e], Wu[e], Wd[e])
        for (sg, su, sd) in shared:                           # shared experts last
            y += ffn(X[b], sg, su, sd)
        Y[b] = y
    return Y, ids_out, p_out
