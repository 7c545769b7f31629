"""CPU oracle for the verification step of judge speculative decoding.  TEST INFRASTRUCTURE.

This file is the plain, slow, fp64 statement of what one verification step computes:
the target decoder's forward over the block ``[x_t, d_1 .. d_gamma]`` against an existing
KV cache (Eq. 2), the probability-ratio acceptance test (Eq. 3) or its temperature-0
form (strict / greedy matching), the judge verifier score on the hidden state of each
drafted token (Eq. 4, Eq. 5), the either-test-accepts rule (Sec. 3.2, App. D.2), the
accept-until-first-rejection scan (Sec. 3.1), the token emitted after the accepted prefix
and the resulting cache length.

Also here, for the calls built around the step: the top-k alignment baseline of the paper's
experiments (Sec. 4) and the semantic-preservation score that labels the verifier's training
tokens (Sec. 3.3, Eq. 6 in the autoregressive form of Eq. 7).

It is independent of the CUDA library: it imports nothing from it, shares no helper,
table or constant with it, and is only ever called from tests, the smoke check and the
benchmark's CPU-baseline leg.  numpy's matmul is the only library primitive used; there
is no tiling, fusion or reordering beyond what the definitions state.

Parity status.  Every function below is pinned by tests that do not re-use its own
formulae (an independent decoder implementation, closed forms, brute force on tiny
inputs, Monte-Carlo distribution tests).  One thing is *parity unpinned*: the behaviour
of a verifier trained on the paper's labels (accepted-length statistics of Table 1 / 2);
the verifier weights are an input here.

Conventions (row j = 0..gamma of a sequence's block):
  * row 0's input token is the pending token x_t (not yet in the cache); row j >= 1 is d_j;
  * row j sits at absolute position L + j, L = number of cached tokens;
  * logits of row j give the target distribution p_{j+1} for drafted position j+1
    (row gamma is the bonus distribution);
  * the judge input for d_j is the final-norm hidden state of row j.
"""
from __future__ import annotations

import dataclasses
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64

# --------------------------------------------------------------------------------------
# decoder pieces (the model family the paper evaluates: RMSNorm, RoPE, GQA, SwiGLU)
# --------------------------------------------------------------------------------------


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x * gain / sqrt(mean(x^2) + eps), row-wise."""
    x = np.asarray(x, F64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(gain, F64)


def rope(x: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing.

    x: [rows, heads, hd].  Pair (i, i + hd/2) is rotated by angle pos * theta^(-2i/hd).
    """
    x = np.asarray(x, F64)
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = theta ** (-(2.0 * np.arange(half, dtype=F64)) / hd)
    ang = np.asarray(positions, F64)[:, None] * inv_freq[None, :]          # [rows, half]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def softmax_rows(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, F64)
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)


@dataclasses.dataclass
class Shape:
    """Decoder dimensions (the oracle keeps its own copy of the few numbers it needs)."""

    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_theta: float
    rms_eps: float


def attention(q: np.ndarray, k_all: np.ndarray, v_all: np.ndarray, n_cached: int) -> np.ndarray:
    """Causal grouped-query attention of a block over cache + block.

    q:     [rows, Hq, hd]  (already rotated)
    k_all: [n_cached + rows, Hkv, hd]   cache rows followed by the block's own rows
    v_all: same shape.
    Row j sees keys 0 .. n_cached + j (inclusive).  Query head h reads KV head h // (Hq/Hkv).
    Scores are scaled by 1/sqrt(hd); softmax in fp64.
    """
    rows, hq, hd = q.shape
    hkv = k_all.shape[1]
    group = hq // hkv
    out = np.zeros((rows, hq, hd), F64)
    scale = 1.0 / np.sqrt(float(hd))
    for h in range(hq):
        kh = k_all[:, h // group, :]
        vh = v_all[:, h // group, :]
        for j in range(rows):
            n_vis = n_cached + j + 1
            s = (kh[:n_vis] @ q[j, h]) * scale
            s = s - s.max()
            e = np.exp(s)
            out[j, h] = (e / e.sum()) @ vh[:n_vis]
    return out


def layer_forward(x: np.ndarray, w: Dict[str, np.ndarray], cache_k: np.ndarray, cache_v: np.ndarray,
                  shape: Shape) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """One pre-norm decoder layer over a block of rows appended after ``cache_k/v``.

    x: [rows, d] residual stream.  cache_k / cache_v: [L, Hkv, hd] (keys already rotated).
    Matrices are row-major [out, in].  Returns (x_out, k_new [rows,Hkv,hd], v_new).
    """
    rows = x.shape[0]
    L = cache_k.shape[0]
    pos = L + np.arange(rows)
    a = rmsnorm(x, w["norm_attn"], shape.rms_eps)
    q = a @ w["wq"].T
    k = a @ w["wk"].T
    v = a @ w["wv"].T
    if "bq" in w and w["bq"] is not None:
        q = q + w["bq"]
        k = k + w["bk"]
        v = v + w["bv"]
    q = rope(q.reshape(rows, shape.n_q_heads, shape.head_dim), pos, shape.rope_theta)
    k = rope(k.reshape(rows, shape.n_kv_heads, shape.head_dim), pos, shape.rope_theta)
    v = v.reshape(rows, shape.n_kv_heads, shape.head_dim)
    k_all = np.concatenate([np.asarray(cache_k, F64), k], axis=0)
    v_all = np.concatenate([np.asarray(cache_v, F64), v], axis=0)
    o = attention(q, k_all, v_all, L).reshape(rows, shape.n_q_heads * shape.head_dim)
    x = x + o @ w["wo"].T
    a = rmsnorm(x, w["norm_ffn"], shape.rms_eps)
    x = x + (silu(a @ w["w_gate"].T) * (a @ w["w_up"].T)) @ w["w_down"].T
    return x, k, v


@dataclasses.dataclass
class BlockForward:
    hidden: np.ndarray           # [rows, d]  after the final norm (LM-head and judge input)
    hidden_pre_norm: np.ndarray  # [rows, d]  residual stream after the last layer
    logits: np.ndarray           # [rows, V]
    k_new: List[np.ndarray]      # per layer [rows, Hkv, hd]
    v_new: List[np.ndarray]


def forward_blocks(shape: Shape, top: Dict[str, np.ndarray], layer_provider: Callable[[int], Dict[str, np.ndarray]],
                   tokens: Sequence[np.ndarray], caches: Sequence[Sequence[Tuple[np.ndarray, np.ndarray]]]
                   ) -> List[BlockForward]:
    """Target forward over one block per sequence (Eq. 2), layers outermost.

    tokens[b]: int array [rows_b] = [x_t, d_1..d_gamma].  caches[b][layer] = (K [L_b,Hkv,hd], V).
    ``layer_provider(l)`` returns layer l's fp64 tensors; it is called once per layer so that
    large models can be streamed.  Sequences are independent of one another.
    """
    emb = top["embed"]
    xs = [np.asarray(emb[np.asarray(t, np.int64)], F64) for t in tokens]
    k_new = [[] for _ in tokens]
    v_new = [[] for _ in tokens]
    for l in range(shape.n_layers):
        w = layer_provider(l)
        for b in range(len(tokens)):
            ck, cv = caches[b][l]
            xs[b], k, v = layer_forward(xs[b], w, ck, cv, shape)
            k_new[b].append(k)
            v_new[b].append(v)
        del w
    out = []
    for b in range(len(tokens)):
        h = rmsnorm(xs[b], top["final_norm"], shape.rms_eps)
        logits = h @ np.asarray(top["lm_head"], F64).T
        out.append(BlockForward(h, xs[b], logits, k_new[b], v_new[b]))
    return out


def prefill(shape: Shape, top, layer_provider, tokens: np.ndarray):
    """Full causal forward from an empty cache; returns (BlockForward, cache list)."""
    empty = [(np.zeros((0, shape.n_kv_heads, shape.head_dim)), np.zeros((0, shape.n_kv_heads, shape.head_dim)))
             for _ in range(shape.n_layers)]
    bf = forward_blocks(shape, top, layer_provider, [tokens], [empty])[0]
    return bf, list(zip(bf.k_new, bf.v_new))


# --------------------------------------------------------------------------------------
# verification rule
# --------------------------------------------------------------------------------------


def judge_scores(hidden_rows: np.ndarray, w: np.ndarray, b: float) -> np.ndarray:
    """Verifier(h) = sigmoid(w . h + b): logistic regression on the hidden state (Eq. 5)."""
    z = np.asarray(hidden_rows, F64) @ np.asarray(w, F64) + float(b)
    return 1.0 / (1.0 + np.exp(-z))


GREEDY, SAMPLING = 0, 1


def argmax_lowest(row: np.ndarray) -> int:
    """Index of the maximum; the lowest index wins ties."""
    return int(np.argmax(row))


@dataclasses.dataclass
class Verdict:
    accepted_len: int
    next_token: int
    new_kv_len: int
    judge: np.ndarray        # [gamma] sigmoid scores s_1..s_gamma
    p_draft: np.ndarray      # [gamma] p_j(d_j) (softmax(logits/T) of row j-1 at token d_j)
    align: np.ndarray        # [gamma] bool: alignment test alone
    judge_ok: np.ndarray     # [gamma] bool: judge test alone
    accept: np.ndarray       # [gamma] bool: final per-position bit
    margins: Dict[str, np.ndarray]  # quantities a comparison needs to spot near-ties


def verdict(logits: np.ndarray, hidden: np.ndarray, draft_ids: np.ndarray, n_cached: int, *,
            mode: int, temperature: float = 1.0, q_tok: Optional[np.ndarray] = None,
            q_full: Optional[np.ndarray] = None, uniforms: Optional[np.ndarray] = None,
            judge_w: Optional[np.ndarray] = None, judge_b: float = 0.0, theta: float = 0.5,
            use_align: bool = True, use_judge: bool = True, top_k: int = 1) -> Verdict:
    """Acceptance decision for one sequence from the block's logits and hidden states.

    logits [gamma+1, V], hidden [gamma+1, d] (rows as in the module docstring),
    draft_ids [gamma], q_tok [gamma] = q_j(d_j), q_full [gamma, V], uniforms [gamma+1]
    (entries 0..gamma-1 are u_1..u_gamma of Eq. 3, entry gamma drives the emitted token).

    Decisions that compare floating-point numbers are taken in fp32, the precision the
    compared quantities are handed over in (q and u are fp32 inputs).

    top_k > 1 (greedy mode) relaxes strict matching to the top-k baseline of the paper's experiments
    (Sec. 4): d_j is aligned when it is among the k most likely target tokens, equal logits ranking
    by token id, lowest first.
    """
    gamma = int(len(draft_ids))
    f32 = np.float32
    # judge test: Verifier(h_j) > theta, strict (Eq. 5)
    if judge_w is not None:
        s = judge_scores(hidden[1:gamma + 1], judge_w, judge_b)
    else:
        s = np.zeros(gamma)
    judge_ok = s.astype(f32) > f32(theta)
    # alignment test
    align = np.zeros(gamma, bool)
    p_draft = np.zeros(gamma)
    top_gap = np.zeros(gamma + 1)
    for j in range(gamma + 1):
        srt = np.sort(logits[j])
        top_gap[j] = srt[-1] - srt[-2]
    if mode == GREEDY:
        # strict matching: accept d_j iff it is the target's greedy token (Sec. 3.1)
        p = None
        for j in range(1, gamma + 1):
            if top_k <= 1:
                align[j - 1] = int(draft_ids[j - 1]) == argmax_lowest(logits[j - 1])
            else:
                ranked = np.lexsort((np.arange(logits.shape[1]), -np.asarray(logits[j - 1], F64)))   # by logit, then id
                align[j - 1] = int(draft_ids[j - 1]) in set(int(v) for v in ranked[:top_k])
            p_draft[j - 1] = softmax_rows(logits[j - 1])[int(draft_ids[j - 1])]
    else:
        p = softmax_rows(np.asarray(logits, F64) / float(temperature))
        for j in range(1, gamma + 1):
            pj = p[j - 1, int(draft_ids[j - 1])]
            p_draft[j - 1] = pj
            # u < min(1, p/q)  <=>  u*q < p for q > 0 (u < 1); the product form also
            # covers q == 0 (accept iff p > 0)  -- Eq. 3
            align[j - 1] = f32(uniforms[j - 1]) * f32(q_tok[j - 1]) < f32(pj)
    accept = (align & bool(use_align)) | (judge_ok & bool(use_judge))
    # accept sequentially until the first rejection
    n = 0
    while n < gamma and accept[n]:
        n += 1
    # token emitted after the accepted prefix
    cdf_info = {}
    if mode == GREEDY:
        nxt = argmax_lowest(logits[n])
    else:
        if n < gamma:
            wv = np.maximum(0.0, p[n] - np.asarray(q_full[n], F64))   # residual distribution
            if not wv.sum() > 0.0:
                wv = p[n].copy()
        else:
            wv = p[gamma].copy()                                       # bonus token
        cum = np.cumsum(wv)
        target = float(f32(uniforms[gamma])) * cum[-1]
        nxt = int(np.searchsorted(cum, target, side="right"))          # smallest v with cum[v] > target
        nxt = min(nxt, len(wv) - 1)
        lo = cum[nxt - 1] if nxt > 0 else 0.0
        cdf_info = {"cdf_target": np.array(target), "cdf_lo": np.array(lo), "cdf_hi": np.array(cum[nxt]),
                    "cdf_total": np.array(cum[-1])}
    margins = {"top_gap": top_gap, **cdf_info}
    return Verdict(n, nxt, n_cached + 1 + n, s, p_draft, align, judge_ok, accept, margins)


def verify(shape: Shape, top, layer_provider, pending: Sequence[int], draft_ids: Sequence[np.ndarray],
           caches, *, mode: int, temperature: float = 1.0, q_tok=None, q_full=None, uniforms=None,
           judge_w=None, judge_b: float = 0.0, theta: float = 0.5, use_align=True, use_judge=True
           ) -> Tuple[List[Verdict], List[BlockForward]]:
    """One whole verification step for a batch of independent sequences."""
    tokens = [np.concatenate([[int(pending[b])], np.asarray(draft_ids[b], np.int64)]) for b in range(len(pending))]
    fwd = forward_blocks(shape, top, layer_provider, tokens, caches)
    out = []
    for b, bf in enumerate(fwd):
        out.append(verdict(
            bf.logits, bf.hidden, np.asarray(draft_ids[b]), caches[b][0][0].shape[0], mode=mode,
            temperature=temperature,
            q_tok=None if q_tok is None else q_tok[b], q_full=None if q_full is None else q_full[b],
            uniforms=None if uniforms is None else uniforms[b],
            judge_w=judge_w, judge_b=judge_b, theta=theta, use_align=use_align, use_judge=use_judge))
    return out, fwd


# --------------------------------------------------------------------------------------
# semantic-preservation score (labels for the verifier's training data)
# --------------------------------------------------------------------------------------


def log_softmax_rows(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, F64)
    z = z - z.max(axis=-1, keepdims=True)
    return z - np.log(np.exp(z).sum(axis=-1, keepdims=True))


def teacher_forced_logp(shape: Shape, top, layer_provider, cache, prev_token: int, tokens: Sequence[int]) -> np.ndarray:
    """log P(tokens[k] | cache, prev_token, tokens[:k]) for every k: one block [prev_token, tokens...] fed to the
    target (Eq. 2), row k's distribution read at tokens[k]."""
    block = np.concatenate([[int(prev_token)], np.asarray(tokens, np.int64)])
    bf = forward_blocks(shape, top, layer_provider, [block], [cache])[0]
    lp = log_softmax_rows(bf.logits)
    return np.array([lp[k, int(tokens[k])] for k in range(len(tokens))])


def semantic_preservation_score(shape: Shape, top, layer_provider, cache, prev_token: int, y_i: int, z_i: int,
                                future: Sequence[int]) -> Tuple[float, float]:
    """s(y, z_i) of Sec. 3.3 with N = len(future) future tokens (Eq. 6, in the autoregressive form of Eq. 7):

        s = [log P(z_i | y_<i) - log P(y_i | y_<i)]
            + sum_k [log P(y_{i+k} | y_<i, z_i, y_{i+1..i+k-1}) - log P(y_{i+k} | y_<i, y_i, y_{i+1..i+k-1})]

    cache holds y_{<i-1}, prev_token is y_{i-1} (the row that predicts position i), future = y_{i+1..i+N}.
    The replaced-token probabilities come from feeding the token-substituted response to the target.
    Returns (s, s_prefix)."""
    lp_z = teacher_forced_logp(shape, top, layer_provider, cache, prev_token, [int(z_i)] + [int(t) for t in future])
    lp_y = teacher_forced_logp(shape, top, layer_provider, cache, prev_token, [int(y_i)] + [int(t) for t in future])
    return float(np.sum(lp_z - lp_y)), float(lp_z[0] - lp_y[0])
