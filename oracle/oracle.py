"""ctypes front end of the CPU oracle (``corun_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, ``__graft_entry__.smoke()`` and
the ``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``.  It shares no
code with the CUDA path and never imports it.

The functions mirror the paper's notation: a request is a prompt ``x`` plus a
seed ``s`` (Design, "Determinism Contract"); prefill produces the first token,
each decode step one more (Background, "LLM Inference and Continuous Batching");
``variate_u24`` is R(s, t) and ``sample`` is S ("Determinism Argument").
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "corun_oracle.c")
_LIB = os.path.join(_HERE, "libcorun_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math) and return the path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=gnu11", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab")] + [
        ("rms_eps", C.c_float), ("rope_theta", C.c_float)]


_PP = C.POINTER(C.c_void_p)


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", _PP), ("wqkv", _PP), ("wo", _PP),
                ("mlp_norm", _PP), ("wgate_up", _PP), ("wdown", _PP)]


class _Moe(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_experts", "top_k", "expert_ffn", "n_shared", "renormalize")] + [
        ("router", _PP), ("gate_up", _PP), ("down", _PP)]


class _Mla(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kv_lora_rank", "qk_nope", "qk_rope", "v_head", "first_dense")] + [
        ("kv_norm", _PP), ("wkv_b", _PP)]


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_forward.restype = C.c_int
        L.orc_forward.argtypes = [C.POINTER(_Shape), C.POINTER(_Weights), C.c_void_p, C.c_int64, C.c_int64,
                                  C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int]
        L.orc_forward_ex.restype = C.c_int
        L.orc_forward_ex.argtypes = [C.POINTER(_Shape), C.POINTER(_Weights), C.POINTER(_Moe), C.c_void_p, C.c_int64,
                                     C.c_int64, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int]
        L.orc_forward_mla.restype = C.c_int
        L.orc_forward_mla.argtypes = [C.POINTER(_Shape), C.POINTER(_Weights), C.POINTER(_Mla), C.POINTER(_Moe), C.c_void_p,
                                      C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int]
        L.orc_mla_attention.restype = None
        L.orc_mla_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64] + [C.c_int32] * 5 + [C.c_void_p, C.c_void_p]
        L.orc_moe_ffn.restype = None
        L.orc_moe_ffn.argtypes = [C.POINTER(_Moe), C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_matmul_bf16.restype = None
        L.orc_matmul_bf16.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p]
        L.orc_rmsnorm.restype = None
        L.orc_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_float, C.c_void_p]
        L.orc_rope.restype = None
        L.orc_rope.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.c_float]
        L.orc_silu.restype = C.c_double
        L.orc_silu.argtypes = [C.c_double]
        L.orc_attention.restype = None
        L.orc_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                    C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        L.orc_philox4x32_10.restype = None
        L.orc_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_variate_u24.restype = C.c_uint32
        L.orc_variate_u24.argtypes = [C.c_uint64, C.c_uint64]
        L.orc_sample.restype = C.c_int32
        L.orc_sample.argtypes = [C.c_void_p, C.c_int64, C.c_float, C.c_float, C.c_uint32, C.POINTER(C.c_double)]
        L.orc_sample_plain.restype = C.c_int32
        L.orc_sample_plain.argtypes = [C.c_void_p, C.c_int64, C.c_float, C.c_float, C.c_uint32, C.POINTER(C.c_double)]
        L.orc_sample_plain_many.restype = None
        L.orc_sample_plain_many.argtypes = [C.c_void_p, C.c_int64, C.c_float, C.c_float, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
        L.orc_sample_many.restype = None
        L.orc_sample_many.argtypes = [C.c_void_p, C.c_int64, C.c_float, C.c_float, C.c_void_p, C.c_int64, C.c_void_p]
        L.orc_num_threads.restype = C.c_int
        L.orc_weight.restype = C.c_uint64
        L.orc_weight.argtypes = [C.c_float, C.c_float, C.c_float]
        _lib = L
    return _lib


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "weights are bf16 bit patterns (uint16)"
    return a


@dataclass
class Shape:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0


class Model:
    """Weights of one decoder as bf16 bit patterns (numpy uint16), borrowed.

    ``weights`` keys: embed [V,H], lm_head [V,H], final_norm [H], and lists of
    L arrays: attn_norm [H], wqkv [(nq+2nkv)*hd, H] (q rows, then k, then v),
    wo [H, nq*hd], mlp_norm [H], wgate_up [2F, H] (gate rows, then up), wdown [H, F].

    ``moe`` (optional) turns every feed-forward layer into a Mixture-of-Experts block: a dict with
    n_experts, top_k, expert_ffn, n_shared, renormalize and lists of L arrays router [E, H],
    gate_up [(E+S)*2F, H] (block e = expert e: gate rows then up rows), down [H, (E+S)*F]; the dense
    wgate_up / wdown entries are then unused (any placeholders).
    """

    def __init__(self, shape: Shape, weights: dict, moe: dict = None, mla: dict = None):
        self.shape = shape
        self.mla = None
        self._keep = {k: ([_u16(x) for x in v] if isinstance(v, (list, tuple)) else _u16(v))
                      for k, v in weights.items()}
        sh = shape
        self._cs = _Shape(sh.n_layers, sh.hidden, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.ffn, sh.vocab,
                          sh.rms_eps, sh.rope_theta)
        self._arrs = {}
        cw = _Weights()
        for k in ("embed", "lm_head", "final_norm"):
            setattr(cw, k, _ptr(self._keep[k]))
        for k in ("attn_norm", "wqkv", "wo", "mlp_norm", "wgate_up", "wdown"):
            arr = (C.c_void_p * sh.n_layers)(*[_ptr(x) for x in self._keep[k]])
            self._arrs[k] = arr
            setattr(cw, k, C.cast(arr, _PP))
        self._cw = cw
        self._cm = None
        if moe is not None:
            self._moe_keep = {k: [_u16(x) for x in moe[k]] for k in ("router", "gate_up", "down")}
            cm = _Moe(moe["n_experts"], moe["top_k"], moe["expert_ffn"], moe["n_shared"], 1 if moe.get("renormalize") else 0)
            for k in ("router", "gate_up", "down"):
                arr = (C.c_void_p * sh.n_layers)(*[_ptr(x) for x in self._moe_keep[k]])
                self._arrs["moe_" + k] = arr
                setattr(cm, k, C.cast(arr, _PP))
            self._cm = cm
            self.moe = dict(moe)

        if mla is not None:
            # MLA decoder: wqkv is [nh*(nope+rope) + rank + rope, H], wo [H, nh*v]; kv_norm L x [rank], wkv_b L x
            # [nh*(nope+v), rank]; layers below first_dense are dense (wgate_up / wdown), the others MoE
            self._mla_keep = {k: [_u16(x) for x in mla[k]] for k in ("kv_norm", "wkv_b")}
            cl = _Mla(mla["kv_lora_rank"], mla["qk_nope"], mla["qk_rope"], mla["v_head"], mla["first_dense"])
            for k in ("kv_norm", "wkv_b"):
                arr = (C.c_void_p * sh.n_layers)(*[_ptr(x) for x in self._mla_keep[k]])
                self._arrs["mla_" + k] = arr
                setattr(cl, k, C.cast(arr, _PP))
            self._cl = cl
            self.mla = dict(mla)

    def moe_ffn_row(self, layer: int, x):
        """One row through the Mixture-of-Experts block of ``layer``: (y [H], ids [top_k], weights [top_k])."""
        x = _f32(x)
        y = np.empty_like(x)
        k = self.moe["top_k"]
        ids = np.zeros(k, np.int32)
        pr = np.zeros(k, np.float64)
        lib().orc_moe_ffn(C.byref(self._cm), layer, x.shape[0], _ptr(x), _ptr(y), _ptr(ids), _ptr(pr))
        return y, ids, pr

    def new_cache(self, max_T: int):
        sh = self.shape
        if self.mla is not None:                        # one latent + rotary key per token and layer
            return (np.zeros((sh.n_layers, max_T, self.mla["kv_lora_rank"] + self.mla["qk_rope"]), np.float32), None)
        kd = sh.n_kv_heads * sh.head_dim
        return (np.zeros((sh.n_layers, max_T, kd), np.float32), np.zeros((sh.n_layers, max_T, kd), np.float32))

    def forward(self, tokens, pos0: int, cache, want: str = "last"):
        """Run ``tokens`` of one request at positions pos0.. ; returns logits.

        want: "last" -> [V]; "all" -> [T, V]; "none" -> None (cache fill only).
        """
        K, V = cache
        toks = np.ascontiguousarray(tokens, dtype=np.int32)
        T = toks.shape[0]
        out = None
        if want == "all":
            out = np.empty((T, self.shape.vocab), np.float32)
        elif want == "last":
            out = np.empty((self.shape.vocab,), np.float32)
        if self.mla is not None:
            rc = lib().orc_forward_mla(C.byref(self._cs), C.byref(self._cw), C.byref(self._cl),
                                       C.byref(self._cm) if self._cm is not None else None, _ptr(toks), T, pos0, _ptr(K),
                                       K.shape[1], _ptr(out) if out is not None else None, 1 if want == "all" else 0)
        else:
            rc = lib().orc_forward_ex(C.byref(self._cs), C.byref(self._cw), C.byref(self._cm) if self._cm is not None else None,
                                      _ptr(toks), T, pos0, _ptr(K), _ptr(V), K.shape[1],
                                      _ptr(out) if out is not None else None, 1 if want == "all" else 0)
        if rc != 0:
            raise ValueError("orc_forward: bad argument")
        return out


class Request:
    """State z_t of one request: prompt + generated prefix, its cache, its seed."""

    def __init__(self, model: Model, prompt, seed: int, temperature: float = 0.0, top_p: float = 1.0,
                 max_T: int = 0):
        self.model, self.seed, self.temperature, self.top_p = model, int(seed), float(temperature), float(top_p)
        self.prompt = list(int(t) for t in prompt)
        self.cache = model.new_cache(max_T or (len(self.prompt) + 64))
        self.n_ctx = 0          # tokens cached
        self.t = 0              # generation step
        self.pending = None     # token to feed next
        self.logits = None

    def prefill(self):
        self.logits = self.model.forward(self.prompt, 0, self.cache)
        self.n_ctx = len(self.prompt)
        return self._sample()

    def decode(self, force_token=None):
        tok = self.pending if force_token is None else int(force_token)
        self.logits = self.model.forward([tok], self.n_ctx, self.cache)
        self.n_ctx += 1
        return self._sample()

    def _sample(self):
        tok, _ = sample(self.logits, self.temperature, self.top_p, variate_u24(self.seed, self.t))
        self.t += 1
        self.pending = tok
        return tok


def forward_rows(model: Model, rows):
    """Batched entry: ``rows`` is a list of (tokens, pos0, cache) of independent
    requests; each is evaluated by itself, in order.  Exists so that the
    row-independence pin has something to exercise."""
    return [model.forward(t, p, c) for (t, p, c) in rows]


def matmul_bf16(W_bits, X):
    W_bits = _u16(W_bits)
    X = _f32(X)
    R, K = X.shape
    N = W_bits.shape[0]
    out = np.empty((R, N), np.float32)
    lib().orc_matmul_bf16(_ptr(W_bits), N, K, _ptr(X), R, _ptr(out))
    return out


def rmsnorm(x, g_bits, eps):
    x = _f32(x)
    out = np.empty_like(x)
    g_bits = _u16(g_bits)
    lib().orc_rmsnorm(_ptr(x), _ptr(g_bits), x.shape[0], eps, _ptr(out))
    return out


def rope(v, pos: int, theta: float):
    v = _f32(v).copy()
    lib().orc_rope(_ptr(v), v.shape[0], pos, theta)
    return v


def silu(z: float) -> float:
    return lib().orc_silu(z)


def attention(q, K, V, p: int):
    """q [nq, hd]; K, V [T, nkv, hd] with T > p; causal over 0..p."""
    q, K, V = _f32(q), _f32(K), _f32(V)
    nq, hd = q.shape
    nkv = K.shape[1]
    out = np.empty((nq, hd), np.float32)
    lib().orc_attention(_ptr(q), _ptr(K), _ptr(V), nkv * hd, p, nq, nkv, hd, _ptr(out))
    return out


def philox4x32_10(ctr, key):
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    o = np.empty(4, np.uint32)
    lib().orc_philox4x32_10(_ptr(c), _ptr(k), _ptr(o))
    return o


def variate_u24(seed: int, t: int) -> int:
    return int(lib().orc_variate_u24(seed & (2**64 - 1), t))


def sample(logits, temperature: float, top_p: float, u24: int):
    """S(logits, u): returns (token, margin)."""
    lg = _f32(logits)
    m = C.c_double(0.0)
    tok = lib().orc_sample(_ptr(lg), lg.shape[0], temperature, top_p, u24, C.byref(m))
    return int(tok), float(m.value)


def sample_plain(logits, temperature: float, top_p: float, u24: int):
    """The plain fp64 definition of S (the pin of the integer specification): returns (token, margin)."""
    lg = _f32(logits)
    m = C.c_double(0.0)
    tok = lib().orc_sample_plain(_ptr(lg), lg.shape[0], temperature, top_p, u24, C.byref(m))
    return int(tok), float(m.value)


def sample_plain_many(logits, temperature: float, top_p: float, u24s):
    """Plain S for many variates against one row: (tokens int32[n], margins float64[n])."""
    lg = _f32(logits)
    u = np.ascontiguousarray(u24s, dtype=np.uint32)
    tok = np.empty(u.shape[0], np.int32)
    mg = np.empty(u.shape[0], np.float64)
    lib().orc_sample_plain_many(_ptr(lg), lg.shape[0], temperature, top_p, _ptr(u), u.shape[0], _ptr(tok), _ptr(mg))
    return tok, mg


def sample_many(logits, temperature: float, top_p: float, u24s):
    """The integer specification S for many variates against one row (temperature > 0): tokens int32[n]."""
    lg = _f32(logits)
    u = np.ascontiguousarray(u24s, dtype=np.uint32)
    tok = np.empty(u.shape[0], np.int32)
    lib().orc_sample_many(_ptr(lg), lg.shape[0], temperature, top_p, _ptr(u), u.shape[0], _ptr(tok))
    return tok


def weight(logit: float, max_logit: float, inv_t_log2e: float) -> int:
    """Integer sampling weight floor(2^40 * exp2(...)) of one token (see corun_oracle.c)."""
    return int(lib().orc_weight(logit, max_logit, inv_t_log2e))


def num_threads() -> int:
    return int(lib().orc_num_threads())
