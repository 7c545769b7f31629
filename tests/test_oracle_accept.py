"""Pins for the oracle's verification rule (Eq. 3, Eq. 5, either-test-accepts, first rejection)."""
import itertools

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import sj_oracle as orc


def _rand_case(rng, gamma, V, d=16, peaked=True):
    logits = rng.standard_normal((gamma + 1, V)) * (3.0 if peaked else 0.3)
    hidden = rng.standard_normal((gamma + 1, d))
    w = rng.standard_normal(d) / np.sqrt(d)
    return logits, hidden, w


def test_greedy_is_longest_argmax_matching_prefix_brute_force():
    rng = np.random.default_rng(0)
    for trial in range(300):
        gamma, V = int(rng.integers(1, 7)), int(rng.integers(2, 9))
        logits, hidden, w = _rand_case(rng, gamma, V)
        tgt = logits.argmax(axis=1)
        drafts = np.where(rng.random(gamma) < 0.7, tgt[:gamma], rng.integers(0, V, gamma))
        v = orc.verdict(logits, hidden, drafts, 10, mode=orc.GREEDY, judge_w=w, use_judge=False)
        n = 0
        for j in range(gamma):
            if drafts[j] != tgt[j]:
                break
            n += 1
        assert v.accepted_len == n
        assert v.next_token == tgt[n]
        assert v.new_kv_len == 10 + 1 + n
        # with the judge: longest prefix of (match OR score > theta)
        s = scipy.special.expit(hidden[1:] @ w)
        vj = orc.verdict(logits, hidden, drafts, 10, mode=orc.GREEDY, judge_w=w, theta=0.5)
        ok = (drafts == tgt[:gamma]) | (s.astype(np.float32) > np.float32(0.5))
        nj = gamma if ok.all() else int(np.argmin(ok))
        assert vj.accepted_len == nj and vj.next_token == tgt[nj]
        assert np.allclose(vj.judge, s, rtol=0, atol=1e-15)


def test_argmax_ties_take_lowest_index():
    logits = np.array([[1.0, 5.0, 5.0, 2.0], [7.0, 7.0, 7.0, 7.0]])
    hidden = np.zeros((2, 4))
    v = orc.verdict(logits, hidden, np.array([1]), 0, mode=orc.GREEDY)
    assert v.accepted_len == 1 and v.next_token == 0
    v = orc.verdict(logits, hidden, np.array([2]), 0, mode=orc.GREEDY)
    assert v.accepted_len == 0 and v.next_token == 1


def test_or_truth_table_and_flags():
    # one drafted position; make (align, judge) take all four values
    V, d = 4, 3
    for align, judge in itertools.product([False, True], repeat=2):
        logits = np.zeros((2, V)); logits[0, 2] = 5.0
        draft = np.array([2 if align else 1])
        hidden = np.zeros((2, d)); hidden[1, 0] = 4.0 if judge else -4.0
        w = np.array([1.0, 0, 0])
        for ua, uj in itertools.product([False, True], repeat=2):
            v = orc.verdict(logits, hidden, draft, 0, mode=orc.GREEDY, judge_w=w, theta=0.5,
                            use_align=ua, use_judge=uj)
            assert v.accepted_len == int((align and ua) or (judge and uj))
            assert bool(v.align[0]) == align and bool(v.judge_ok[0]) == judge


def test_threshold_limits_and_monotonicity_and_two_stage_dominates():
    rng = np.random.default_rng(1)
    for trial in range(200):
        gamma, V = int(rng.integers(1, 9)), 6
        logits, hidden, w = _rand_case(rng, gamma, V)
        drafts = rng.integers(0, V, gamma)
        q = rng.dirichlet(np.ones(V), gamma)
        u = rng.random(gamma + 1).astype(np.float32)
        for mode in (orc.GREEDY, orc.SAMPLING):
            kw = dict(mode=mode, q_tok=q[np.arange(gamma), drafts], q_full=q, uniforms=u, judge_w=w)
            off = orc.verdict(logits, hidden, drafts, 0, use_judge=False, **kw)
            t0 = orc.verdict(logits, hidden, drafts, 0, theta=0.0, **kw)
            t1 = orc.verdict(logits, hidden, drafts, 0, theta=1.0, **kw)
            assert t0.accepted_len == gamma                      # sigmoid > 0 always
            assert (t1.accepted_len, t1.next_token) == (off.accepted_len, off.next_token)
            prev = gamma
            for th in (0.1, 0.3, 0.5, 0.7, 0.9):
                n = orc.verdict(logits, hidden, drafts, 0, theta=th, **kw).accepted_len
                assert n <= prev
                prev = n
            two = orc.verdict(logits, hidden, drafts, 0, theta=0.5, **kw).accepted_len
            jo = orc.verdict(logits, hidden, drafts, 0, theta=0.5, use_align=False, **kw).accepted_len
            assert two >= max(off.accepted_len, jo)


def test_sampling_accept_bit_is_eq3_including_q_zero():
    # u < min(1, p/q), evaluated by hand
    logits = np.log(np.array([[0.5, 0.25, 0.25], [1 / 3, 1 / 3, 1 / 3]]))
    hidden = np.zeros((2, 2))
    for q_tok, u, want in [(0.25, 0.99, True),     # p=0.5 > q  -> ratio 1
                           (1.0, 0.49, True),      # ratio 0.5, u below
                           (1.0, 0.51, False),     # ratio 0.5, u above
                           (0.0, 0.99, True)]:     # q = 0 < p: always accepted
        qf = np.array([[q_tok, (1 - q_tok) / 2, (1 - q_tok) / 2]])
        v = orc.verdict(logits, hidden, np.array([0]), 0, mode=orc.SAMPLING, q_tok=np.array([q_tok]),
                        q_full=qf, uniforms=np.array([u, 0.3], np.float32))
        assert bool(v.align[0]) == want
        assert np.isclose(v.p_draft[0], 0.5)


def test_residual_and_bonus_inverse_cdf_by_hand():
    p = np.array([0.1, 0.6, 0.3]); q = np.array([0.5, 0.2, 0.3])
    logits = np.log(np.stack([p, np.array([0.2, 0.3, 0.5])]))
    hidden = np.zeros((2, 2))
    # draft token 0: p/q = 0.2; u = 0.9 rejects; residual = max(0,p-q) = [0, .4, 0] -> token 1
    for ur in (0.0, 0.5, 0.999):
        v = orc.verdict(logits, hidden, np.array([0]), 0, mode=orc.SAMPLING, q_tok=q[[0]], q_full=q[None],
                        uniforms=np.array([0.9, ur], np.float32))
        assert (v.accepted_len, v.next_token) == (0, 1)
    # accepted (u = 0.1): bonus from row 1 = [.2,.3,.5] by inverse CDF
    for ur, tok in [(0.0, 0), (0.19, 0), (0.21, 1), (0.49, 1), (0.51, 2), (0.999, 2)]:
        v = orc.verdict(logits, hidden, np.array([0]), 0, mode=orc.SAMPLING, q_tok=q[[0]], q_full=q[None],
                        uniforms=np.array([0.1, ur], np.float32))
        assert (v.accepted_len, v.next_token) == (1, tok)
    # temperature: softmax(logits / T); T -> 0 concentrates on the argmax
    v = orc.verdict(logits, hidden, np.array([0]), 0, mode=orc.SAMPLING, temperature=0.01, q_tok=q[[0]],
                    q_full=q[None], uniforms=np.array([0.9, 0.7], np.float32))
    assert v.next_token == 1 and v.p_draft[0] < 1e-50


@pytest.mark.parametrize("V", [4, 13, 64])
def test_sampling_reproduces_target_distribution_monte_carlo(V):
    """Judge off: the first emitted token is distributed as p_1 (Eq. 3 + residual resampling),
    the acceptance rate is sum_v min(p_v, q_v), and after a full accept the bonus token ~ p_{gamma+1}."""
    rng = np.random.default_rng(100 + V)
    gamma = 2
    logits = rng.standard_normal((gamma + 1, V)) * 1.5
    p = orc.softmax_rows(logits)
    q = rng.dirichlet(np.full(V, 0.5), gamma)
    hidden = np.zeros((gamma + 1, 2))
    N = 120_000
    first = np.zeros(V); bonus = np.zeros(V); acc0 = 0; full = 0
    drafts_all = np.stack([rng.choice(V, size=N, p=q[j]) for j in range(gamma)], axis=1)
    us = rng.random((N, gamma + 1)).astype(np.float32)
    for t in range(N):
        d = drafts_all[t]
        v = orc.verdict(logits, hidden, d, 0, mode=orc.SAMPLING, q_tok=q[np.arange(gamma), d], q_full=q,
                        uniforms=us[t], use_judge=False)
        if v.accepted_len >= 1:
            acc0 += 1
            first[d[0]] += 1
        else:
            first[v.next_token] += 1
        if v.accepted_len == gamma:
            full += 1
            bonus[v.next_token] += 1
    # acceptance rate of position 1 against the closed form
    a = np.minimum(p[0], q[0]).sum()
    assert abs(acc0 / N - a) < 4 * np.sqrt(a * (1 - a) / N)
    chi = scipy.stats.chisquare(first, p[0] * N)
    assert chi.pvalue > 1e-3, chi
    chi_b = scipy.stats.chisquare(bonus, p[gamma] * full)
    assert chi_b.pvalue > 1e-3, chi_b


def test_judge_score_closed_form():
    rng = np.random.default_rng(7)
    h = rng.standard_normal((5, 32)); w = rng.standard_normal(32); b = 0.37
    assert np.allclose(orc.judge_scores(h, w, b), scipy.special.expit(h @ w + b), rtol=1e-14, atol=0)
    assert orc.judge_scores(np.zeros((1, 32)), w, 0.0)[0] == 0.5


def test_residual_with_zero_mass_falls_back_to_the_target_distribution():
    """p == q at the rejected position (here both exactly uniform): max(0, p - q) has no mass, so the emitted
    token is drawn from p itself.  With u = 0.6 over four equally likely tokens the inverse CDF gives token 2;
    an all-zero weight vector would instead run off the end (token 3)."""
    V = 4
    logits = np.zeros((2, V))                       # softmax: exactly 0.25 each
    hidden = np.zeros((2, 3))
    q_full = np.full((1, V), 0.25)
    # the scalar q handed over for the drafted token is larger than p, so u * q >= p rejects position 1
    v = orc.verdict(logits, hidden, np.array([1]), 5, mode=orc.SAMPLING, temperature=1.0, q_tok=np.array([1.0]),
                    q_full=q_full, uniforms=np.array([0.99, 0.6]), use_judge=False)
    assert v.accepted_len == 0 and v.next_token == 2 and v.new_kv_len == 6
    for u, tok in [(0.0, 0), (0.2499, 0), (0.25, 1), (0.74, 2), (0.76, 3)]:
        v = orc.verdict(logits, hidden, np.array([1]), 5, mode=orc.SAMPLING, q_tok=np.array([1.0]), q_full=q_full,
                        uniforms=np.array([0.99, u]), use_judge=False)
        assert v.next_token == tok
    # q above p everywhere it matters (q puts all its mass on one token the target gives 1/4): the residual is
    # p on the other three tokens, renormalised; u = 0.5 lands on the middle one of them
    q_full = np.array([[0.0, 1.0, 0.0, 0.0]])
    v = orc.verdict(logits, hidden, np.array([1]), 5, mode=orc.SAMPLING, q_tok=np.array([1.0]), q_full=q_full,
                    uniforms=np.array([0.99, 0.5]), use_judge=False)
    assert v.accepted_len == 0 and v.next_token == 2


def test_top_k_alignment_is_rank_below_k_brute_force():
    """Top-k baseline (Sec. 4): a draft is aligned iff fewer than k tokens rank before it, a token ranking before
    another when its logit is larger or equal with a lower id.  k = 1 is strict matching."""
    rng = np.random.default_rng(5)
    for trial in range(200):
        gamma, V = int(rng.integers(1, 6)), int(rng.integers(3, 10))
        logits = np.round(rng.standard_normal((gamma + 1, V)) * 2.0) / 2.0      # coarse values: many exact ties
        hidden = np.zeros((gamma + 1, 4))
        drafts = rng.integers(0, V, gamma)
        for k in (1, 2, 3):
            v = orc.verdict(logits, hidden, drafts, 3, mode=orc.GREEDY, use_judge=False, top_k=k)
            n = 0
            for j in range(gamma):
                d = int(drafts[j])
                before = sum(1 for t in range(V) if t != d and (logits[j, t] > logits[j, d] or (logits[j, t] == logits[j, d] and t < d)))
                if before >= k:
                    break
                n += 1
            assert v.accepted_len == n, (trial, k)
            assert v.next_token == int(np.argmax(logits[n]))
        strict = orc.verdict(logits, hidden, drafts, 3, mode=orc.GREEDY, use_judge=False)
        assert strict.accepted_len == orc.verdict(logits, hidden, drafts, 3, mode=orc.GREEDY, use_judge=False, top_k=1).accepted_len
