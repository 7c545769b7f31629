"""Pins for the oracle's decoder forward (Eq. 2, Eq. 4): an independent implementation,
library attention, and self-consistency between cached and uncached evaluation."""
import numpy as np
import pytest
import torch

import helpers
from oracle import sj_oracle as orc
from paper_2510_02329_b200 import synth


def _hf_logits_hidden(shape: synth.ModelShape, model: helpers.HostModel, tokens: np.ndarray):
    """The same random-init decoder evaluated by the installed transformers implementation, fp64."""
    if shape.qkv_bias:
        from transformers import Qwen2Config as Cfg, Qwen2ForCausalLM as LM
        extra = {}
    else:
        from transformers import LlamaConfig as Cfg, LlamaForCausalLM as LM
        extra = {"attention_bias": False, "mlp_bias": False, "head_dim": shape.head_dim}
    cfg = Cfg(vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.d_ffn,
              num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_q_heads,
              num_key_value_heads=shape.n_kv_heads, rms_norm_eps=shape.rms_eps,
              rope_parameters={"rope_type": "default", "rope_theta": shape.rope_theta},
              tie_word_embeddings=shape.tied_embeddings, max_position_embeddings=4096,
              attn_implementation="eager", **extra)
    lm = LM(cfg).to(torch.float64).eval()
    sd = {"model.embed_tokens.weight": model.top["embed"], "model.norm.weight": model.top["final_norm"],
          "lm_head.weight": model.top["lm_head"]}
    names = {"wq": "self_attn.q_proj.weight", "wk": "self_attn.k_proj.weight", "wv": "self_attn.v_proj.weight",
             "wo": "self_attn.o_proj.weight", "w_gate": "mlp.gate_proj.weight", "w_up": "mlp.up_proj.weight",
             "w_down": "mlp.down_proj.weight", "norm_attn": "input_layernorm.weight",
             "norm_ffn": "post_attention_layernorm.weight", "bq": "self_attn.q_proj.bias",
             "bk": "self_attn.k_proj.bias", "bv": "self_attn.v_proj.bias"}
    for l, lw in enumerate(model.layers):
        for k, v in lw.items():
            sd[f"model.layers.{l}.{names[k]}"] = v
    missing, unexpected = lm.load_state_dict({k: v.to(torch.float64) for k, v in sd.items()}, strict=False)
    assert not unexpected, unexpected
    assert all("rotary" in m or "inv_freq" in m for m in missing), missing
    assert lm.config.head_dim == shape.head_dim if hasattr(lm.config, "head_dim") else True
    with torch.no_grad():
        out = lm(torch.from_numpy(tokens.astype(np.int64))[None], output_hidden_states=True)
    return out.logits[0].numpy(), out


SHAPES = [
    synth.TINY,                                                                    # MHA, hd 64
    synth.ModelShape("gqa", 2, 128, 8, 2, 16, 320, 512, rope_theta=5e5),            # GQA group 4
    synth.ModelShape("gqa-hd-free", 2, 96, 4, 2, 32, 256, 300, rope_theta=1e4),     # Hq*hd != d
    synth.ModelShape("qwen-bias", 2, 128, 4, 2, 32, 256, 400, rope_theta=1e6, qkv_bias=True),
    synth.ModelShape("tied", 1, 64, 2, 1, 32, 128, 200, tied_embeddings=True),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: s.name)
def test_cached_block_matches_independent_decoder(shape):
    """Oracle prefill + cached block forward == transformers' decoder on the whole sequence."""
    model = helpers.HostModel(shape, torch.float32)
    L, gamma = 37, 5
    toks = synth.token_ids(shape.vocab, L + 1 + gamma, seed=3)
    ref_logits, _ = _hf_logits_hidden(shape, model, toks)
    osh = helpers.oracle_shape(shape)
    top = model.top64()
    _, cache = orc.prefill(osh, top, model.layer64, toks[:L])
    bf = orc.forward_blocks(osh, top, model.layer64, [toks[L:]], [cache])[0]
    # the library evaluates its rotary table in fp32, which bounds the agreement at ~1e-7;
    # any structural mistake (pairing, sign, head mapping, norm placement) is O(1)
    scale = np.abs(ref_logits).max()
    assert np.abs(bf.logits - ref_logits[L:]).max() <= 2e-6 * max(1.0, scale)


def test_cached_equals_full_recompute_and_single_row_decode():
    shape = SHAPES[1]
    model = helpers.HostModel(shape, torch.float32)
    osh, top = helpers.oracle_shape(shape), model.top64()
    toks = synth.token_ids(shape.vocab, 30, seed=5)
    full, full_cache = orc.prefill(osh, top, model.layer64, toks)
    _, cache = orc.prefill(osh, top, model.layer64, toks[:21])
    blk = orc.forward_blocks(osh, top, model.layer64, [toks[21:]], [cache])[0]
    assert np.abs(blk.logits - full.logits[21:]).max() < 1e-10
    assert np.abs(blk.hidden - full.hidden[21:]).max() < 1e-10
    for l in range(shape.n_layers):
        assert np.abs(blk.k_new[l] - full_cache[l][0][21:]).max() < 1e-12
        assert np.abs(blk.v_new[l] - full_cache[l][1][21:]).max() < 1e-12
    # gamma = 0: a block of one row is an ordinary decode step
    _, cache29 = orc.prefill(osh, top, model.layer64, toks[:29])
    one = orc.forward_blocks(osh, top, model.layer64, [toks[29:]], [cache29])[0]
    assert np.abs(one.logits[0] - full.logits[29]).max() < 1e-10


def test_attention_against_library_sdpa():
    rng = np.random.default_rng(0)
    rows, L, hq, hkv, hd = 5, 19, 6, 2, 16
    q = rng.standard_normal((rows, hq, hd))
    k = rng.standard_normal((L + rows, hkv, hd))
    v = rng.standard_normal((L + rows, hkv, hd))
    got = orc.attention(q, k, v, L)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(hq // hkv, 0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(hq // hkv, 0)[None]
    mask = torch.ones(rows, L + rows, dtype=torch.bool).tril(diagonal=L)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask)[0].permute(1, 0, 2).numpy()
    assert np.abs(got - ref).max() < 1e-12


def test_rope_is_a_position_dependent_rotation():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((4, 3, 8))
    pos = np.array([0, 1, 7, 1000])
    y = orc.rope(x, pos, 1e4)
    assert np.allclose(y[0], x[0])                                   # position 0: identity
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1))
    # relative-position property: <rope(a,m), rope(b,n)> depends on m-n only
    a, b = rng.standard_normal((1, 1, 8)), rng.standard_normal((1, 1, 8))
    d1 = (orc.rope(a, [5], 1e4) * orc.rope(b, [2], 1e4)).sum()
    d2 = (orc.rope(a, [105], 1e4) * orc.rope(b, [102], 1e4)).sum()
    assert abs(d1 - d2) < 1e-9
    # explicit 2x2 rotation of pair (i, i+hd/2), i = 1, angle = pos * theta^(-2i/hd)
    ang = 7 * 1e4 ** (-2 * 1 / 8)
    assert np.isclose(y[2, 0, 1], x[2, 0, 1] * np.cos(ang) - x[2, 0, 5] * np.sin(ang))
    assert np.isclose(y[2, 0, 5], x[2, 0, 5] * np.cos(ang) + x[2, 0, 1] * np.sin(ang))


def test_rmsnorm_softmax_silu_closed_forms():
    x = np.array([[3.0, -4.0]])
    assert np.allclose(orc.rmsnorm(x, np.array([2.0, 0.5]), 0.0), [[2 * 3 / np.sqrt(12.5), -0.5 * 4 / np.sqrt(12.5)]])
    p = orc.softmax_rows(np.array([[0.0, np.log(3.0)], [1000.0, 1000.0]]))
    assert np.allclose(p, [[0.25, 0.75], [0.5, 0.5]])
    assert np.isclose(orc.silu(np.array([0.0, 2.0]))[1], 2.0 / (1 + np.exp(-2.0)))
