"""Seeded synthetic inputs for the verification step (shapes, sizes, value distributions).

This module only *draws inputs*: model shapes, random-init weights, KV-cache fills, token
ids, draft probabilities and uniforms.  It contains none of the method's arithmetic (no
transformer layer, no softmax, no acceptance rule) and is the one module that both the
CPU oracle's tests and the CUDA path's tests/bench are allowed to share.

Weights and cache fills come from a counter-based generator (a splitmix64-style hash of
``(seed, tensor_id, element index)`` followed by Box-Muller in fp64), so any slice of any
tensor can be drawn on any torch device without holding the whole model anywhere.  The
bytes handed to the oracle and to the GPU are always the *same* bytes: a tensor is drawn
once, rounded once to its storage dtype, and then copied, never re-drawn per side.

Small per-step inputs (token ids, Dirichlet draft probabilities, uniforms) use numpy's
Philox generator on the host.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import numpy as np
import torch

# --------------------------------------------------------------------------------------
# model shapes
# --------------------------------------------------------------------------------------


@dataclasses.dataclass(frozen=True)
class ModelShape:
    """Decoder shape; names follow the usual Llama/Qwen config vocabulary."""

    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_theta: float = 1e4
    rms_eps: float = 1e-5
    tied_embeddings: bool = False
    qkv_bias: bool = False

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def layer_params(self) -> int:
        d = self.d_model
        return d * self.q_dim + 2 * d * self.kv_dim + self.q_dim * d + 3 * d * self.d_ffn

    def streamed_params(self) -> int:
        """Parameters read once per verify step (layers + LM head; norms ignored)."""
        return self.n_layers * self.layer_params() + self.vocab * self.d_model

    def kv_bytes_per_token(self, elem_bytes: int = 2) -> int:
        return self.n_layers * 2 * self.kv_dim * elem_bytes

    def cut(self, n_layers: int, vocab: Optional[int] = None, name: Optional[str] = None) -> "ModelShape":
        """Same widths, fewer layers (and optionally a smaller vocab): parity-test cuts."""
        return dataclasses.replace(
            self, n_layers=n_layers, vocab=vocab or self.vocab, name=name or f"{self.name}-cut{n_layers}"
        )


TINY = ModelShape("tiny", 2, 256, 4, 4, 64, 1024, 4096, rope_theta=1e4)
LLAMA_1B = ModelShape("llama-3.2-1b-shaped", 16, 2048, 32, 8, 64, 8192, 128256, rope_theta=5e5,
                      tied_embeddings=True)
LLAMA_8B = ModelShape("llama-3.1-8b-shaped", 32, 4096, 32, 8, 128, 14336, 128256, rope_theta=5e5)
QWEN_32B = ModelShape("qwen2.5-32b-shaped", 64, 5120, 40, 8, 128, 27648, 152064, rope_theta=1e6,
                      qkv_bias=True)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration: a shape plus batch, cache length and gamma."""

    name: str
    shape: ModelShape
    batch: int
    gamma: int
    kv_len: int            # fixed length, or upper bound when ragged
    kv_len_min: int = 0    # >0: lengths drawn uniformly in [kv_len_min, kv_len]
    page_size: int = 16
    draft_match_prob: float = 0.0  # >0: drafts follow the target argmax with this probability


WORKLOADS: Dict[str, Workload] = {
    "cfg1": Workload("cfg1-tiny-b1-kv128-g4", TINY, 1, 4, 128),
    "cfg2": Workload("cfg2-1b-b1-kv2048-g8", LLAMA_1B, 1, 8, 2048),
    "cfg3": Workload("cfg3-8b-b1-kv4096-g8", LLAMA_8B, 1, 8, 4096),
    "cfg3-g4": Workload("cfg3-8b-b1-kv4096-g4", LLAMA_8B, 1, 4, 4096),
    "cfg3-g16": Workload("cfg3-8b-b1-kv4096-g16", LLAMA_8B, 1, 16, 4096),
    "cfg4": Workload("cfg4-8b-b32-ragged512-8192-g8", LLAMA_8B, 32, 8, 8192, kv_len_min=512,
                     draft_match_prob=0.6),
    "cfg5": Workload("cfg5-32b-b8-kv8192-g8", QWEN_32B, 8, 8, 8192),
}

# --------------------------------------------------------------------------------------
# counter-based generator
# --------------------------------------------------------------------------------------

_M64 = (1 << 64) - 1


def _s64(c: int) -> int:
    """Python int -> the signed 64-bit value with the same bit pattern."""
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)
_GOLD = _s64(0x9E3779B97F4A7C15)
_ODD = _s64(0x632BE59BD9B4E019)


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    """Logical right shift on int64 tensors (torch's >> is arithmetic)."""
    return (x >> k) & ((1 << (64 - k)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    return x ^ _lsr(x, 31)


def _mix_int(x: int) -> int:
    x &= _M64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _M64
    return x ^ (x >> 31)


def tensor_key(seed: int, *ids: int) -> int:
    """Fold a seed and a tuple of small integers (tensor kind, layer, ...) into a 64-bit key."""
    k = _mix_int(seed + 0x1234567)
    for i in ids:
        k = _mix_int(k ^ ((i + 1) * 0x9E3779B97F4A7C15))
    return k


_CHUNK = 1 << 22


def _std_normal_range(key: int, start: int, count: int, device) -> torch.Tensor:
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    base = (idx * _GOLD) ^ _s64(key)
    h1 = _mix(base)
    h2 = _mix(base + _ODD)
    u1 = (_lsr(h1, 11).to(torch.float64) + 0.5) * (2.0 ** -53)
    u2 = (_lsr(h2, 11).to(torch.float64) + 0.5) * (2.0 ** -53)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def normal(key: int, shape, std: float, dtype: torch.dtype, device="cpu", start: int = 0) -> torch.Tensor:
    """``N(0, std^2)`` tensor of the given shape, element ``i`` a pure function of ``(key, start+i)``."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    for off in range(0, n, _CHUNK):
        c = min(_CHUNK, n - off)
        out[off:off + c] = (_std_normal_range(key, start + off, c, device) * std).to(dtype)
    return out.view(*shape)


# tensor kinds (first id after the seed)
K_EMBED, K_LMHEAD, K_WQ, K_WK, K_WV, K_WO, K_WG, K_WU, K_WD, K_BQ, K_BK, K_BV, K_JUDGE, K_CACHE_K, K_CACHE_V = range(15)

_LAYER_KINDS = {
    "wq": K_WQ, "wk": K_WK, "wv": K_WV, "wo": K_WO, "w_gate": K_WG, "w_up": K_WU, "w_down": K_WD,
    "bq": K_BQ, "bk": K_BK, "bv": K_BV,
}


def layer_tensor_shapes(s: ModelShape) -> Dict[str, tuple]:
    """Row-major ``[out_features, in_features]`` matrices (the nn.Linear convention)."""
    shapes = {
        "wq": (s.q_dim, s.d_model), "wk": (s.kv_dim, s.d_model), "wv": (s.kv_dim, s.d_model),
        "wo": (s.d_model, s.q_dim), "w_gate": (s.d_ffn, s.d_model), "w_up": (s.d_ffn, s.d_model),
        "w_down": (s.d_model, s.d_ffn),
    }
    if s.qkv_bias:
        shapes.update({"bq": (s.q_dim,), "bk": (s.kv_dim,), "bv": (s.kv_dim,)})
    return shapes


WEIGHT_STD = 0.02


def layer_weights(s: ModelShape, layer: int, dtype: torch.dtype, device="cpu", seed: int = 0) -> Dict[str, torch.Tensor]:
    """All tensors of one decoder layer: matrices and biases ``N(0, 0.02^2)``, norm gains 1."""
    out = {}
    for name, shp in layer_tensor_shapes(s).items():
        out[name] = normal(tensor_key(seed, _LAYER_KINDS[name], layer), shp, WEIGHT_STD, dtype, device)
    out["norm_attn"] = torch.ones(s.d_model, dtype=dtype, device=device)
    out["norm_ffn"] = torch.ones(s.d_model, dtype=dtype, device=device)
    return out


def top_weights(s: ModelShape, dtype: torch.dtype, device="cpu", seed: int = 0) -> Dict[str, torch.Tensor]:
    """Embedding, LM head (the same tensor when tied) and the final norm gain."""
    embed = normal(tensor_key(seed, K_EMBED), (s.vocab, s.d_model), WEIGHT_STD, dtype, device)
    if s.tied_embeddings:
        lm_head = embed
    else:
        lm_head = normal(tensor_key(seed, K_LMHEAD), (s.vocab, s.d_model), WEIGHT_STD, dtype, device)
    return {"embed": embed, "lm_head": lm_head, "final_norm": torch.ones(s.d_model, dtype=dtype, device=device)}


def judge_head(s: ModelShape, device="cpu", seed: int = 0) -> torch.Tensor:
    """Verifier weight ``w ~ N(0, 1/d)`` in fp32 (bias 0 in every configuration)."""
    return normal(tensor_key(seed, K_JUDGE), (s.d_model,), 1.0 / math.sqrt(s.d_model), torch.float32, device)


def cache_fill(s: ModelShape, layer: int, seq: int, n_tokens: int, dtype: torch.dtype, device="cpu",
               seed: int = 0, std_k: Optional[float] = None, std_v: Optional[float] = None):
    """Synthetic cache rows ``[n_tokens, n_kv_heads, head_dim]`` for K (post-RoPE) and V.

    The cache is an *input* of the verification step; for the large shapes it is drawn
    directly at the scale a prefill of the same random-init model produces (the projections
    of a unit-RMS vector through ``N(0, 0.02^2)`` weights have std ``0.02 * sqrt(d)``).
    """
    sd = WEIGHT_STD * math.sqrt(s.d_model)
    k = normal(tensor_key(seed, K_CACHE_K, layer, seq), (n_tokens, s.n_kv_heads, s.head_dim),
               std_k if std_k is not None else sd, dtype, device)
    v = normal(tensor_key(seed, K_CACHE_V, layer, seq), (n_tokens, s.n_kv_heads, s.head_dim),
               std_v if std_v is not None else sd, dtype, device)
    return k, v


# --------------------------------------------------------------------------------------
# per-step inputs (host, numpy Philox)
# --------------------------------------------------------------------------------------


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & _M64, stream]))


def token_ids(vocab: int, n: int, seed: int = 0, stream: int = 1) -> np.ndarray:
    return _rng(seed, stream).integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


def kv_lengths(w: Workload, seed: int = 0) -> np.ndarray:
    if w.kv_len_min > 0:
        return _rng(seed, 2).integers(w.kv_len_min, w.kv_len + 1, size=w.batch).astype(np.int32)
    return np.full(w.batch, w.kv_len, dtype=np.int32)


def dirichlet_rows(n_rows: int, vocab: int, alpha: float = 0.1, seed: int = 0, stream: int = 3) -> np.ndarray:
    """``n_rows`` draws of Dirichlet(alpha * 1_V), stored fp32 (tiny entries underflow to 0)."""
    g = _rng(seed, stream)
    out = np.empty((n_rows, vocab), dtype=np.float32)
    for r in range(n_rows):
        x = g.standard_gamma(alpha, size=vocab)
        tot = x.sum()
        out[r] = (x / tot).astype(np.float32)
    return out


def uniforms(shape, seed: int = 0, stream: int = 4) -> np.ndarray:
    """fp32 uniforms in [0, 1)."""
    u = _rng(seed, stream).random(size=shape, dtype=np.float32)
    return np.minimum(u, np.float32(1.0 - 2.0 ** -24))


def page_permutation(n_pages: int, seed: int = 0, stream: int = 5) -> np.ndarray:
    return _rng(seed, stream).permutation(n_pages).astype(np.int32)


@dataclasses.dataclass
class StepInputs:
    pending: np.ndarray        # [B] int32   token x_t fed at row 0
    draft_ids: np.ndarray      # [B, gamma] int32
    draft_q_full: np.ndarray   # [B, gamma, V] fp32
    draft_q_tok: np.ndarray    # [B, gamma] fp32   q_j(d_j)
    uniforms: np.ndarray       # [B, gamma+1] fp32


def step_inputs(vocab: int, batch: int, gamma: int, seed: int = 0, draft_ids: Optional[np.ndarray] = None) -> StepInputs:
    pend = token_ids(vocab, batch, seed, stream=11)
    if draft_ids is None:
        draft_ids = token_ids(vocab, batch * gamma, seed, stream=12).reshape(batch, gamma)
    qf = dirichlet_rows(batch * gamma, vocab, 0.1, seed, stream=13).reshape(batch, gamma, vocab)
    qt = np.take_along_axis(qf, draft_ids[..., None].astype(np.int64), axis=2)[..., 0].copy()
    u = uniforms((batch, gamma + 1), seed, stream=14)
    return StepInputs(pend, np.ascontiguousarray(draft_ids, dtype=np.int32), qf, qt, u)
