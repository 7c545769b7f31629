"""Pins for the oracle's semantic-preservation score (Sec. 3.3, Eq. 6-7)."""
import numpy as np
import torch

import helpers
from oracle import sj_oracle as orc
from paper_2510_02329_b200 import synth

SHAPE = synth.ModelShape("score-tiny", 2, 64, 4, 2, 16, 128, 97, rope_theta=1e4)


def _model():
    m = helpers.HostModel(SHAPE, torch.float32, "cpu", seed=3)
    return helpers.oracle_shape(SHAPE), m.top64(), m.layer64


def _joint_logp(osh, top, layers, seq):
    """log P(seq[1:] | seq[0]) by one causal forward from an empty cache: the chain rule written out."""
    bf, _ = orc.prefill(osh, top, layers, np.asarray(seq))
    z = bf.logits - bf.logits.max(axis=1, keepdims=True)
    lp = z - np.log(np.exp(z).sum(axis=1, keepdims=True))
    return float(sum(lp[k, seq[k + 1]] for k in range(len(seq) - 1)))


def test_score_is_the_difference_of_joint_log_likelihoods():
    """Eq. 7's telescoping: s(y, z_i) = log P(y_<i, z_i, y_>i) - log P(y_<i, y_i, y_>i); the prefix's own
    likelihood cancels.  The joint likelihoods come from full recomputes, the score from cached blocks."""
    osh, top, layers = _model()
    rng = np.random.default_rng(0)
    for trial in range(4):
        L, N = int(rng.integers(2, 9)), int(rng.integers(0, 6))
        y = rng.integers(0, SHAPE.vocab, L + 1 + N)          # y_0 .. y_{L-1} | y_i | future
        z = int(rng.integers(0, SHAPE.vocab))
        prefix, y_i, future = y[:L], int(y[L]), y[L + 1:]
        _, cache = orc.prefill(osh, top, layers, prefix[:-1])   # cache = y_{<i-1}; y_{i-1} is fed with the block
        s, s_prefix = orc.semantic_preservation_score(osh, top, layers, cache, int(prefix[-1]), y_i, z, future)
        joint_z = _joint_logp(osh, top, layers, np.concatenate([prefix, [z], future]))
        joint_y = _joint_logp(osh, top, layers, np.concatenate([prefix, [y_i], future]))
        assert abs(s - (joint_z - joint_y)) < 1e-9
        # the prefix term alone: N = 0
        s0, s0_prefix = orc.semantic_preservation_score(osh, top, layers, cache, int(prefix[-1]), y_i, z, [])
        assert abs(s0 - s0_prefix) < 1e-12 and abs(s_prefix - s0_prefix) < 1e-12


def test_score_of_the_original_token_is_zero_and_scores_are_antisymmetric():
    osh, top, layers = _model()
    toks = synth.token_ids(SHAPE.vocab, 12, seed=5)
    _, cache = orc.prefill(osh, top, layers, toks[:5])
    s, sp = orc.semantic_preservation_score(osh, top, layers, cache, int(toks[5]), int(toks[6]), int(toks[6]), toks[7:])
    assert s == 0.0 and sp == 0.0
    a, _ = orc.semantic_preservation_score(osh, top, layers, cache, int(toks[5]), 11, 40, toks[7:])
    b, _ = orc.semantic_preservation_score(osh, top, layers, cache, int(toks[5]), 40, 11, toks[7:])
    assert abs(a + b) < 1e-12


def test_teacher_forced_logp_rows_are_log_probabilities():
    osh, top, layers = _model()
    toks = synth.token_ids(SHAPE.vocab, 9, seed=6)
    _, cache = orc.prefill(osh, top, layers, toks[:3])
    lp = orc.teacher_forced_logp(osh, top, layers, cache, int(toks[3]), toks[4:])
    assert (lp < 0).all()
    # summing exp over every possible first token gives 1
    tot = sum(np.exp(orc.teacher_forced_logp(osh, top, layers, cache, int(toks[3]), [v])[0]) for v in range(SHAPE.vocab))
    assert abs(tot - 1.0) < 1e-12
