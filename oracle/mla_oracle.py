"""Plain CPU oracle of multi-head latent attention (MLA) for one query token at decode time.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``.  No CUDA kernel for it exists yet; the oracle and its
pins come first.  It shares no code with the CUDA path.

What it computes (the paper evaluates an MLA model -- Evaluation, "Setup" -- and names its attention
backend in the throughput discussion, without formulas; this is the standard definition at the
DeepSeek-V2-Lite shape the workload names: latent width d_c = 512, rope width d_r = 64, per-head
no-rope width d_n = 128 and value width d_v = 128).  Per cached token t the cache holds the latent
c_t [d_c] and the shared rotary key r_t [d_r] (already rotated); per head h there are up-projections
W_uk[h] [d_n, d_c] and W_uv[h] [d_v, d_c]:

    k_{h,t} = [ W_uk[h] c_t ; r_t ]              v_{h,t} = W_uv[h] c_t
    s_{h,t} = ( q_nope[h] . W_uk[h] c_t + q_rope[h] . r_t ) / sqrt(d_n + d_r)
    p_h     = softmax_t(s_{h,.})                 o_h = sum_t p_{h,t} v_{h,t}

``attend`` is this definition written out (keys and values decompressed, then ordinary attention);
``attend_absorbed`` is the algebraically equal form a decode kernel uses, which never decompresses:
q_lat[h] = W_uk[h]^T q_nope[h], s_{h,t} = (q_lat[h] . c_t + q_rope[h] . r_t) / sqrt(d_n + d_r),
o_h = W_uv[h] (sum_t p_{h,t} c_t).  Everything is fp64, positions in ascending order.

Pins (tests/test_mla_oracle.py): the two forms against each other, the definition against a library
attention routine on the decompressed keys and values, a hand-computed two-token example, one cached
token (the output is that token's value whatever the query), and invariance to a joint orthogonal change
of basis of the latent space.
"""
from __future__ import annotations

import numpy as np


def _softmax(s: np.ndarray) -> np.ndarray:
    z = np.exp(s - s.max())
    return z / z.sum()


def attend(q_nope, q_rope, C, Rk, W_uk, W_uv) -> np.ndarray:
    """q_nope [n_heads, d_n], q_rope [n_heads, d_r]; cache C [T, d_c], Rk [T, d_r]; W_uk [n_heads, d_n, d_c],
    W_uv [n_heads, d_v, d_c].  Returns o [n_heads, d_v]."""
    q_nope, q_rope, C, Rk = (np.asarray(a, dtype=np.float64) for a in (q_nope, q_rope, C, Rk))
    W_uk, W_uv = np.asarray(W_uk, dtype=np.float64), np.asarray(W_uv, dtype=np.float64)
    n_heads, d_n = q_nope.shape
    d_r = q_rope.shape[1]
    T = C.shape[0]
    out = np.zeros((n_heads, W_uv.shape[1]))
    for h in range(n_heads):
        s = np.zeros(T)
        V = np.zeros((T, W_uv.shape[1]))
        for t in range(T):
            k_nope = W_uk[h] @ C[t]
            s[t] = (q_nope[h] @ k_nope + q_rope[h] @ Rk[t]) / np.sqrt(d_n + d_r)
            V[t] = W_uv[h] @ C[t]
        p = _softmax(s)
        for t in range(T):
            out[h] += p[t] * V[t]
    return out


def attend_absorbed(q_nope, q_rope, C, Rk, W_uk, W_uv) -> np.ndarray:
    """The same result without decompressing the cache (the form a decode kernel computes)."""
    q_nope, q_rope, C, Rk = (np.asarray(a, dtype=np.float64) for a in (q_nope, q_rope, C, Rk))
    W_uk, W_uv = np.asarray(W_uk, dtype=np.float64), np.asarray(W_uv, dtype=np.float64)
    n_heads, d_n = q_nope.shape
    d_r = q_rope.shape[1]
    out = np.zeros((n_heads, W_uv.shape[1]))
    for h in range(n_heads):
        q_lat = W_uk[h].T @ q_nope[h]                       # [d_c]
        s = (C @ q_lat + Rk @ q_rope[h]) / np.sqrt(d_n + d_r)
        p = _softmax(s)
        out[h] = W_uv[h] @ (p @ C)
    return out
