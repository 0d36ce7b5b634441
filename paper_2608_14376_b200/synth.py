"""Seeded synthetic inputs: model shapes, weights, prompts, context lengths.

Holds none of the method's arithmetic.  Both the CUDA path's callers and the
CPU oracle's callers take their inputs from here, as bytes.

Recipe (the benchmark configurations): every matrix (embedding, projections, LM head) is
N(0, 0.02) drawn in fp32 and rounded to bf16 (round to nearest even); RMSNorm
gains are 1; prompts are i.i.d. uniform token ids; request seed = 1000 + index.
Tensor draw order: embed, then per layer wqkv, wo, wgate_up, wdown, then lm_head.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0

    def dict(self):
        return asdict(self)

    @property
    def q_dim(self):
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self):
        return self.n_kv_heads * self.head_dim

    @property
    def qkv_dim(self):
        return self.q_dim + 2 * self.kv_dim

    def weight_bytes_per_step(self) -> int:
        """bf16 bytes of every projection + LM head (what one decode step streams)."""
        per_layer = self.qkv_dim * self.hidden + self.hidden * self.q_dim + 2 * self.ffn * self.hidden \
            + self.hidden * self.ffn
        return 2 * (self.n_layers * per_layer + self.vocab * self.hidden)

    def kv_bytes_per_token(self, elem_bytes: int = 2) -> int:
        return 2 * self.kv_dim * elem_bytes * self.n_layers

    def flops_per_row(self) -> int:
        return self.weight_bytes_per_step()  # 2 flop per bf16 weight = its byte count


TINY = ModelShape(2, 256, 4, 2, 64, 768, 2048, 1e-6, 10000.0)
QWEN3_8B = ModelShape(36, 4096, 32, 8, 128, 12288, 151936, 1e-6, 1000000.0)
# Qwen3-30B-A3B-shaped Mixture-of-Experts decoder: 48 layers, hidden 2048, 32 q / 4 kv heads of 128, 128 experts
# of 768 (top-8, renormalised, no shared expert).  `ffn` of the attention shape is a placeholder (the dense
# feed-forward weights are not made); QWEN3_30B_A3B_EFF carries the feed-forward width the row program sees,
# (E + S) * F, for byte counts.
QWEN3_30B_A3B = ModelShape(48, 2048, 32, 4, 128, 64, 151936, 1e-6, 1000000.0)
QWEN3_30B_A3B_MOE = dict(n_experts=128, top_k=8, expert_ffn=768, n_shared=0, renormalize=True)
QWEN3_30B_A3B_EFF = ModelShape(48, 2048, 32, 4, 128, 128 * 768, 151936, 1e-6, 1000000.0)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even (format conversion only)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u >> 16) & 1) + 0x7FFF
    return ((u + r) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def _tensor_list(sh: ModelShape):
    yield "embed", None, (sh.vocab, sh.hidden)
    for l in range(sh.n_layers):
        yield "wqkv", l, (sh.qkv_dim, sh.hidden)
        yield "wo", l, (sh.hidden, sh.q_dim)
        yield "wgate_up", l, (2 * sh.ffn, sh.hidden)
        yield "wdown", l, (sh.hidden, sh.ffn)
    yield "lm_head", None, (sh.vocab, sh.hidden)


def make_weights_numpy(sh: ModelShape, seed: int = 0, std: float = 0.02) -> dict:
    """Weights as numpy uint16 (bf16 bits); for shapes small enough for the host."""
    rng = np.random.Generator(np.random.PCG64(seed))
    w = {"attn_norm": [], "mlp_norm": [], "wqkv": [], "wo": [], "wgate_up": [], "wdown": []}
    one = f32_to_bf16_bits(np.ones(sh.hidden, np.float32))
    for name, l, shape in _tensor_list(sh):
        t = f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))
        if l is None:
            w[name] = t
        else:
            w[name].append(t)
    w["final_norm"] = one.copy()
    for _ in range(sh.n_layers):
        w["attn_norm"].append(one.copy())
        w["mlp_norm"].append(one.copy())
    return w


def make_weights_torch(sh: ModelShape, seed: int = 0, std: float = 0.02, device="cuda", dense_ffn: bool = True) -> dict:
    """Weights as torch bf16 tensors drawn on ``device`` (same recipe; the
    stream differs from the numpy one, so use one generator per experiment).
    ``dense_ffn`` False leaves out wgate_up / wdown (Mixture-of-Experts models bring their own)."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(seed)
    w = {"attn_norm": [], "mlp_norm": [], "wqkv": [], "wo": [], "wgate_up": [], "wdown": []}
    for name, l, shape in _tensor_list(sh):
        if not dense_ffn and name in ("wgate_up", "wdown"):
            continue
        t = torch.empty(shape, dtype=torch.bfloat16, device=device)
        rows = max(1, (1 << 27) // shape[1])  # draw in slabs so the fp32 staging stays small
        for r0 in range(0, shape[0], rows):
            r1 = min(shape[0], r0 + rows)
            t[r0:r1] = (torch.randn((r1 - r0, shape[1]), generator=g, device=device, dtype=torch.float32) * std
                        ).to(torch.bfloat16)
        if l is None:
            w[name] = t
        else:
            w[name].append(t)
    w["final_norm"] = torch.ones(sh.hidden, dtype=torch.bfloat16, device=device)
    for _ in range(sh.n_layers):
        w["attn_norm"].append(torch.ones(sh.hidden, dtype=torch.bfloat16, device=device))
        w["mlp_norm"].append(torch.ones(sh.hidden, dtype=torch.bfloat16, device=device))
    return w


def weights_numpy_to_torch(w: dict, device="cuda") -> dict:
    import torch

    def cv(a):
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)

    return {k: ([cv(x) for x in v] if isinstance(v, list) else cv(v)) for k, v in w.items()}


def weights_torch_to_numpy(w: dict) -> dict:
    import torch

    def cv(t):
        return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)

    return {k: ([cv(x) for x in v] if isinstance(v, list) else cv(v)) for k, v in w.items()}


def make_moe_numpy(sh: ModelShape, n_experts: int, top_k: int, expert_ffn: int, n_shared: int, renormalize: bool = False,
                   seed: int = 0, std: float = 0.02, router_std: float = 0.2) -> dict:
    """Mixture-of-Experts feed-forward layers as numpy uint16 (bf16 bits): per layer router [E, H],
    gate_up [(E+S)*2F, H] (block e = expert e: gate rows then up rows) and down [H, (E+S)*F]."""
    rng = np.random.Generator(np.random.PCG64(seed + 77))
    nb = n_experts + n_shared
    m = dict(n_experts=n_experts, top_k=top_k, expert_ffn=expert_ffn, n_shared=n_shared, renormalize=renormalize,
             router=[], gate_up=[], down=[])
    for _ in range(sh.n_layers):
        m["router"].append(f32_to_bf16_bits(rng.standard_normal((n_experts, sh.hidden), dtype=np.float32) * np.float32(router_std)))
        m["gate_up"].append(f32_to_bf16_bits(rng.standard_normal((nb * 2 * expert_ffn, sh.hidden), dtype=np.float32) * np.float32(std)))
        m["down"].append(f32_to_bf16_bits(rng.standard_normal((sh.hidden, nb * expert_ffn), dtype=np.float32) * np.float32(std)))
    return m


def moe_numpy_to_torch(m: dict, device="cuda") -> dict:
    import torch

    def cv(a):
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)

    return {k: ([cv(x) for x in v] if isinstance(v, list) else v) for k, v in m.items()}


def make_moe_torch(sh: ModelShape, n_experts: int, top_k: int, expert_ffn: int, n_shared: int, renormalize: bool = False,
                   seed: int = 0, std: float = 0.02, router_std: float = 0.2, device="cuda") -> dict:
    """The same layers drawn on the device (for shapes too large for the host)."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(seed + 77)
    nb = n_experts + n_shared
    m = dict(n_experts=n_experts, top_k=top_k, expert_ffn=expert_ffn, n_shared=n_shared, renormalize=renormalize,
             router=[], gate_up=[], down=[])

    def draw(shape, sd):
        t = torch.empty(shape, dtype=torch.bfloat16, device=device)
        rows = max(1, (1 << 27) // shape[1])
        for r0 in range(0, shape[0], rows):
            r1 = min(shape[0], r0 + rows)
            t[r0:r1] = (torch.randn((r1 - r0, shape[1]), generator=g, device=device, dtype=torch.float32) * sd).to(torch.bfloat16)
        return t

    for _ in range(sh.n_layers):
        m["router"].append(draw((n_experts, sh.hidden), router_std))
        m["gate_up"].append(draw((nb * 2 * expert_ffn, sh.hidden), std))
        m["down"].append(draw((sh.hidden, nb * expert_ffn), std))
    return m


def make_prompts(vocab: int, lengths, seed: int) -> list:
    rng = np.random.Generator(np.random.PCG64(seed))
    return [rng.integers(0, vocab, size=int(n), dtype=np.int64).astype(np.int32) for n in lengths]


def uniform_lengths(lo: int, hi: int, n: int, seed: int) -> np.ndarray:
    """n integers uniform in [lo, hi] inclusive."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(lo, hi + 1, size=n, dtype=np.int64)


def pick_slots(B: int, n_active: int, seed: int) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    return np.sort(rng.permutation(B)[:n_active])


def request_seed(index: int) -> int:
    return 1000 + int(index)


def synthetic_kv(n_tokens: int, kv_dim: int, std: float, seed: int, dtype=np.float16):
    """Seeded K and V rows N(0, std^2), pre-rounded to the cache dtype so that
    both sides hold identical numbers.  Returns fp32 arrays [n_tokens, kv_dim]."""
    rng = np.random.Generator(np.random.PCG64(seed))
    k = (rng.standard_normal((n_tokens, kv_dim), dtype=np.float32) * np.float32(std)).astype(dtype).astype(np.float32)
    v = (rng.standard_normal((n_tokens, kv_dim), dtype=np.float32) * np.float32(std)).astype(dtype).astype(np.float32)
    return k, v


def mla_paged_case(B: int, d_k: int, ctx_lo: int, ctx_hi: int, seed: int, device="cuda", page: int = 16, std: float = 0.5):
    """Seeded paged latent cache on the device for timing: contexts uniform in [ctx_lo, ctx_hi], a pool of exactly the
    pages they need (fp16 N(0, std^2), every position finite) and a block table that scatters every row's pages over
    the pool (a seeded permutation).  Returns (pool [P, page, d_k], block_table int32 [B, max_blocks], ctx int32 [B])."""
    import torch

    ctx = uniform_lengths(ctx_lo, ctx_hi, B, seed=seed).astype(np.int32)
    blocks = -(-ctx // page)
    max_blocks = int(blocks.max())
    n_pages = int(blocks.sum())
    g = torch.Generator(device=device).manual_seed(seed)
    pool = (torch.randn((n_pages, page, d_k), generator=g, device=device) * std).to(torch.float16)
    perm = np.random.Generator(np.random.PCG64(seed)).permutation(n_pages).astype(np.int32)
    table = np.zeros((B, max_blocks), np.int32)
    k = 0
    for b in range(B):
        table[b, :blocks[b]] = perm[k:k + blocks[b]]
        k += int(blocks[b])
    return pool, torch.tensor(table, device=device), torch.tensor(ctx, device=device)
