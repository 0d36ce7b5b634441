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


# DeepSeek-V2-Lite-shaped decoder with multi-head latent attention: 27 layers, hidden 2048, 16 heads, latent 512,
# per-head query 128 (no rope) + 64 (rope), value 128; layer 0 a dense feed-forward of 10944, the others 64 routed
# experts of 1408 (top-6, probabilities as they are) plus 2 shared experts.  n_kv_heads / head_dim are placeholders.
DEEPSEEK_V2_LITE = ModelShape(27, 2048, 16, 16, 128, 10944, 102400, 1e-6, 10000.0)
DEEPSEEK_V2_LITE_MLA = dict(kv_lora_rank=512, qk_nope=128, qk_rope=64, v_head=128, first_dense=1)
DEEPSEEK_V2_LITE_MOE = dict(n_experts=64, top_k=6, expert_ffn=1408, n_shared=2, renormalize=False)


def mla_weight_bytes_per_step(sh: ModelShape, mla: dict, moe: dict) -> int:
    """bf16 bytes of every matrix one decode step of the MLA decoder streams (all experts: none is skipped)."""
    nh, rank, nope, rope, vh = sh.n_q_heads, mla["kv_lora_rank"], mla["qk_nope"], mla["qk_rope"], mla["v_head"]
    attn = (nh * (nope + rope) + rank + rope) * sh.hidden + 2 * nh * (nope + vh) * rank - nh * vh * rank + sh.hidden * nh * vh
    # the key up-projections are read from their transposed copy, W_kv_b once more as a whole for the values
    dense = 3 * sh.ffn * sh.hidden
    nd = mla["first_dense"]
    per_moe = 0
    if moe is not None and nd < sh.n_layers:
        nb = moe["n_experts"] + moe["n_shared"]
        per_moe = moe["n_experts"] * sh.hidden + 3 * nb * moe["expert_ffn"] * sh.hidden
    return 2 * (sh.n_layers * attn + nd * dense + (sh.n_layers - nd) * per_moe + sh.vocab * sh.hidden)


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


def _mla_tensor_list(sh: ModelShape, mla: dict):
    nh, rank, nope, rope, vh = sh.n_q_heads, mla["kv_lora_rank"], mla["qk_nope"], mla["qk_rope"], mla["v_head"]
    yield "embed", None, (sh.vocab, sh.hidden)
    for l in range(sh.n_layers):
        yield "wqkv", l, (nh * (nope + rope) + rank + rope, sh.hidden)
        yield "wkv_b", l, (nh * (nope + vh), rank)
        yield "wo", l, (sh.hidden, nh * vh)
        if l < mla["first_dense"]:
            yield "wgate_up", l, (2 * sh.ffn, sh.hidden)
            yield "wdown", l, (sh.hidden, sh.ffn)
    yield "lm_head", None, (sh.vocab, sh.hidden)


def make_mla_weights_numpy(sh: ModelShape, mla: dict, seed: int = 0, std: float = 0.02):
    """Weights of a decoder with multi-head latent attention as numpy uint16 (bf16 bits): (weights, mla) where
    ``weights`` has the keys of ``make_weights_numpy`` (wqkv [nh*(nope+rope) + rank + rope, H], wo [H, nh*v];
    wgate_up / wdown drawn for the layers below first_dense, one shared dummy array for the others) and ``mla`` is the given dict plus kv_norm
    (ones) and wkv_b [nh*(nope+v), rank] per layer.  Draw order: embed, per layer wqkv, wkv_b, wo (, wgate_up,
    wdown), then lm_head."""
    rng = np.random.Generator(np.random.PCG64(seed))
    w = {"attn_norm": [], "mlp_norm": [], "wqkv": [], "wo": [], "wgate_up": [], "wdown": []}
    m = dict(mla, kv_norm=[], wkv_b=[])
    dummy = np.zeros((1,), np.uint16)
    for name, l, shape in _mla_tensor_list(sh, mla):
        t = f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))
        if l is None:
            w[name] = t
        elif name == "wkv_b":
            m["wkv_b"].append(t)
        else:
            w[name].append(t)
    one = f32_to_bf16_bits(np.ones(sh.hidden, np.float32))
    w["final_norm"] = one.copy()
    for l in range(sh.n_layers):
        w["attn_norm"].append(one.copy())
        w["mlp_norm"].append(one.copy())
        m["kv_norm"].append(f32_to_bf16_bits(np.ones(mla["kv_lora_rank"], np.float32)))
        if l >= mla["first_dense"]:
            w["wgate_up"].append(dummy)
            w["wdown"].append(dummy)
    return w, m


def mla_numpy_to_torch(w: dict, m: dict, device="cuda"):
    """The same as CUDA bf16 tensors; the feed-forward placeholders of expert layers become None."""
    import torch

    def cv(a):
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)

    nd = m["first_dense"]
    wt = {}
    for k, v in w.items():
        if k in ("wgate_up", "wdown"):
            wt[k] = [cv(x) if l < nd else None for l, x in enumerate(v)]
        else:
            wt[k] = [cv(x) for x in v] if isinstance(v, list) else cv(v)
    mt = {k: ([cv(x) for x in v] if isinstance(v, list) else v) for k, v in m.items()}
    return wt, mt


def make_mla_weights_torch(sh: ModelShape, mla: dict, seed: int = 0, std: float = 0.02, device="cuda"):
    """The same recipe drawn on the device (for shapes too large for the host): (weights, mla)."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(seed)
    w = {"attn_norm": [], "mlp_norm": [], "wqkv": [], "wo": [], "wgate_up": [], "wdown": []}
    m = dict(mla, kv_norm=[], wkv_b=[])
    for name, l, shape in _mla_tensor_list(sh, mla):
        t = torch.empty(shape, dtype=torch.bfloat16, device=device)
        rows = max(1, (1 << 27) // shape[1])
        for r0 in range(0, shape[0], rows):
            r1 = min(shape[0], r0 + rows)
            t[r0:r1] = (torch.randn((r1 - r0, shape[1]), generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
        if l is None:
            w[name] = t
        elif name == "wkv_b":
            m["wkv_b"].append(t)
        else:
            w[name].append(t)
    w["final_norm"] = torch.ones(sh.hidden, dtype=torch.bfloat16, device=device)
    for l in range(sh.n_layers):
        w["attn_norm"].append(torch.ones(sh.hidden, dtype=torch.bfloat16, device=device))
        w["mlp_norm"].append(torch.ones(sh.hidden, dtype=torch.bfloat16, device=device))
        m["kv_norm"].append(torch.ones(mla["kv_lora_rank"], dtype=torch.bfloat16, device=device))
        if l >= mla["first_dense"]:
            w["wgate_up"].append(None)
            w["wdown"].append(None)
    return w, m
