"""GPU parity of the calls built around the verification step: chunked prefill (Eq. 2 on known tokens),
per-sequence thresholds and log-probabilities, the top-2 alignment test (Sec. 4's top-k baseline) and the
semantic-preservation score (Eq. 6-7), each against the CPU oracle on the same seeded bytes."""
import numpy as np
import pytest
import torch

import harness
import helpers
from oracle import sj_oracle as orc
from paper_2510_02329_b200 import synth

pytestmark = pytest.mark.gpu

GQA = synth.ModelShape("gqa-small", 3, 256, 4, 2, 64, 512, 1024, rope_theta=5e5)


def _binding():
    from paper_2510_02329_b200 import binding
    return binding


def _empty_case(shape, dtype, n_seqs=1, gamma=4, seed=0, room=200):
    """A target and a cache with `n_seqs` empty sequences and room for `room` tokens each."""
    b = _binding()
    case = harness.Case(shape, dtype, [0] * n_seqs, gamma, seed=seed, cache="fill")
    dev = "cuda"
    top = {k: v.to(dev) for k, v in case.model.top.items()}
    if shape.tied_embeddings:
        top["lm_head"] = top["embed"]
    layers = [{k: v.to(dev) for k, v in lw.items()} for lw in case.model.layers]
    case.target = b.Target(shape, top, layers, max_rows=64)
    case.target.load_judge_head(case.model.judge_w, 0.0, 0.5)
    case.kv = b.KVCache(case.target, n_seqs, n_seqs * (room // 16 + 2))
    case.seq_ids = list(range(n_seqs))
    return case


PREFILL_CASES = [("tiny-f32", synth.TINY, torch.float32), ("tiny-bf16", synth.TINY, torch.bfloat16),
                 ("gqa-bf16", GQA, torch.bfloat16), ("llama-1b-cut2-bf16", synth.LLAMA_1B.cut(2), torch.bfloat16)]


@pytest.mark.parametrize("name,shape,dtype", PREFILL_CASES, ids=[c[0] for c in PREFILL_CASES])
@pytest.mark.parametrize("n_prompt", [77, 33, 1])
def test_prefill_builds_the_cache_the_oracle_prefill_builds(name, shape, dtype, n_prompt):
    """Blocks of up to 32 (24 with four query heads per KV head) tokens, a ragged last block, a lone last token."""
    b = _binding()
    case = _empty_case(shape, dtype)
    try:
        prompt = synth.token_ids(shape.vocab, n_prompt, seed=21, stream=7)
        nxt = case.kv.prefill(0, prompt)
        assert case.kv.lengths([0]) == [n_prompt]
        bf, cache = orc.prefill(case.osh, case.top64, case.model.layer64, prompt)
        tol = harness.tol_for(dtype, float(np.abs(bf.logits).max()))
        for l in range(shape.n_layers):
            k, v = case.kv.read(0, l, 0, n_prompt)
            ek = np.abs(k.cpu().double().numpy() - cache[l][0])
            ev = np.abs(v.cpu().double().numpy() - cache[l][1])
            assert (ek <= tol.delta(cache[l][0])).all() and (ev <= tol.delta(cache[l][1])).all(), (l, ek.max(), ev.max())
        last = bf.logits[-1]
        assert nxt == int(np.argmax(last)) or last.max() - last[nxt] <= 2 * tol.delta(np.abs(last).max())
        # a verification step on top of the prefilled cache, against the oracle on the rows the library stored
        if n_prompt > 1:
            gamma = 4
            si = synth.step_inputs(shape.vocab, 1, gamma, seed=22)
            stored = [tuple(helpers.np64(t) for t in case.kv.read(0, l, 0, n_prompt)) for l in range(shape.n_layers)]
            v2, f2 = orc.verify(case.osh, case.top64, case.model.layer64, [nxt], si.draft_ids, [stored], mode=orc.GREEDY,
                                judge_w=case.judge_w64, theta=0.5)
            out = b.VerifyBuffers(1, gamma, shape.d_model, shape.vocab, debug=True)
            b.verify(case.target, case.kv, [0], torch.from_numpy(si.draft_ids).cuda(), out, commit=False)   # pending = nxt
            case.target.sync()
            err = np.abs(out.dbg_logits.cpu().numpy()[0] - f2[0].logits)
            assert (err <= tol.delta(f2[0].logits)).all(), err.max()
            assert np.abs(out.judge_scores.cpu().numpy()[0] - v2[0].judge).max() <= tol.judge_abs
    finally:
        case.close()


@pytest.mark.parametrize("options", [{"gemm_impl": 1, "step_impl": 1}, {"gemm_impl": 1, "step_impl": 0}, {"gemm_impl": 0}],
                         ids=["persistent", "tcgen05", "cudacore"])
def test_per_sequence_thresholds_and_log_probabilities(options):
    b = _binding()
    thetas = [0.0, 0.5, 1.0, 0.3]
    case = harness.Case(GQA, torch.bfloat16, [20, 33, 7, 48], 6, seed=9).gpu_setup()
    try:
        for k, v in options.items():
            case.target.set_option(k, v)
        fwd = case.oracle_forward()
        case.kv.set_pending(case.seq_ids, case.inputs.pending)
        out = b.VerifyBuffers(case.B, case.gamma, GQA.d_model, GQA.vocab, debug=True)
        b.verify(case.target, case.kv, case.seq_ids, case.d_draft, out, commit=False, theta_per_seq=thetas)
        case.target.sync()
        g = {k: getattr(out, k).cpu().numpy() for k in ("accepted_len", "next_token", "judge_scores", "p_draft", "new_kv_len")}
        g["hidden"], g["logits"] = out.dbg_hidden.cpu().numpy(), out.dbg_logits.cpu().numpy()
        logp = out.logp_draft.cpu().numpy()
        for i, th in enumerate(thetas):      # sequence by sequence: each has its own threshold
            v = orc.verdict(fwd[i].logits, fwd[i].hidden, case.inputs.draft_ids[i], case.kv_lens[i], mode=orc.GREEDY,
                            judge_w=case.judge_w64, theta=th)
            near = np.abs(v.judge - th) <= 1e-3
            if not near.any():
                assert int(g["accepted_len"][i]) == v.accepted_len, (i, th)
            lp = orc.log_softmax_rows(fwd[i].logits)
            want = np.array([lp[j, case.inputs.draft_ids[i][j]] for j in range(case.gamma)])
            assert np.abs(logp[i] - want).max() <= 4e-2 + 2e-2 * np.abs(fwd[i].logits).max()
            assert np.allclose(np.exp(logp[i]), g["p_draft"][i], rtol=1e-4)
        assert int(g["accepted_len"][0]) == case.gamma          # theta 0: a sigmoid is positive
    finally:
        case.close()


SCORE_CASES = [("tiny-f32", synth.TINY, torch.float32, 20), ("gqa-bf16", GQA, torch.bfloat16, 20),
               ("llama-1b-cut2-bf16", synth.LLAMA_1B.cut(2), torch.bfloat16, 20), ("tiny-bf16-n0", synth.TINY, torch.bfloat16, 0)]


@pytest.mark.parametrize("name,shape,dtype,N", SCORE_CASES, ids=[c[0] for c in SCORE_CASES])
def test_semantic_preservation_score(name, shape, dtype, N):
    """N = 20 future tokens as in the paper's implementation details: two teacher-forced blocks of N + 2 rows."""
    case = _empty_case(shape, dtype)
    try:
        toks = synth.token_ids(shape.vocab, 40 + 2 + N, seed=31, stream=8)
        prefix, y_prev, y_i, future = toks[:40], int(toks[40]), int(toks[41]), toks[42:]
        z_i = int((y_i + 17) % shape.vocab)
        case.kv.prefill(0, prefix, want_next=False)
        case.kv.set_pending([0], [y_prev])
        s, s_prefix = case.kv.semantic_score(0, y_i, z_i, future)
        assert case.kv.lengths([0]) == [40]                      # nothing was committed
        stored = [tuple(helpers.np64(t) for t in case.kv.read(0, l, 0, 40)) for l in range(shape.n_layers)]
        want, want_prefix = orc.semantic_preservation_score(case.osh, case.top64, case.model.layer64, stored, y_prev, y_i,
                                                            z_i, future)
        per_term = 1e-4 if dtype == torch.float32 else 2e-2
        assert abs(s_prefix - want_prefix) <= 2 * per_term, (s_prefix, want_prefix)
        assert abs(s - want) <= 2 * per_term * np.sqrt(N + 1) + per_term, (s, want)
        same, _ = case.kv.semantic_score(0, y_i, y_i, future)    # replacing a token by itself changes nothing
        assert same == 0.0
    finally:
        case.close()


@pytest.mark.parametrize("dtype,options", [(torch.float32, {}), (torch.bfloat16, {"gemm_impl": 0}),
                                            (torch.bfloat16, {"gemm_impl": 1, "step_impl": 0}),
                                            (torch.bfloat16, {"gemm_impl": 1, "step_impl": 1})],
                         ids=["f32", "bf16-cudacore", "bf16-tcgen05", "bf16-persistent"])
def test_top_two_alignment(dtype, options):
    """Drafts built from the oracle's own ranking: the target's best token, its second best, its third best, a
    random one.  With top_k = 2 the first two kinds are aligned, the others are not (judge off)."""
    b = _binding()
    gamma = 6
    probe = harness.Case(GQA, dtype, [30, 9, 41], gamma, seed=17)
    # the ranking of row j depends on drafts 1..j only: build the drafts position by position
    kinds = np.array([[0, 1, 0, 1, 2, 0], [1, 1, 1, 0, 0, 3], [0, 0, 2, 0, 0, 0]])   # 0 best, 1 second, 2 third, 3 random
    drafts = probe.inputs.draft_ids.copy()
    caches = [[(helpers.np64(k), helpers.np64(v)) for k, v in seq] for seq in probe.cache_t]
    for j in range(gamma):
        for i in range(3):
            toks = np.concatenate([[int(probe.inputs.pending[i])], drafts[i, :j]])
            row = orc.forward_blocks(probe.osh, probe.top64, probe.model.layer64, [toks], [caches[i]])[0].logits[-1]
            ranked = np.lexsort((np.arange(row.size), -row))
            if kinds[i, j] < 3:
                drafts[i, j] = ranked[kinds[i, j]]
    case = harness.Case(GQA, dtype, [30, 9, 41], gamma, seed=17, draft_ids=drafts).gpu_setup()
    try:
        for k, v in options.items():
            case.target.set_option(k, v)
        fwd = case.oracle_forward()
        tol = harness.tol_for(dtype, float(max(np.abs(f.logits).max() for f in fwd)))
        checked = 0
        for top_k in (1, 2):
            case.kv.set_pending(case.seq_ids, case.inputs.pending)
            out = b.VerifyBuffers(case.B, gamma, GQA.d_model, GQA.vocab, debug=True)
            b.verify(case.target, case.kv, case.seq_ids, case.d_draft, out, commit=False, use_judge=False, top_k=top_k)
            case.target.sync()
            got = out.accepted_len.cpu().numpy()
            glog = out.dbg_logits.cpu().numpy()
            for i in range(3):
                v = orc.verdict(fwd[i].logits, fwd[i].hidden, drafts[i], case.kv_lens[i], mode=orc.GREEDY, use_judge=False,
                                top_k=top_k)
                err = np.abs(glog[i] - fwd[i].logits)
                assert (err <= tol.delta(fwd[i].logits)).all()
                # a decision can only come out differently where the draft's logit is within twice the actual
                # logit error of the boundary between ranks top_k - 1 and top_k
                crisp = True
                for j in range(min(v.accepted_len + 1, gamma)):
                    row = fwd[i].logits[j]
                    srt = np.sort(row)[::-1]
                    zd = row[drafts[i, j]]
                    edge = srt[top_k] if zd >= srt[top_k - 1] else srt[top_k - 1]
                    crisp = crisp and abs(zd - edge) > 2 * err[j].max()
                if crisp:
                    assert int(got[i]) == v.accepted_len, (top_k, i, got, v.accepted_len)
                    checked += 1
        assert checked >= 5
        # the construction itself: with k = 2 sequence 0 stops at its third-best draft, sequence 1 at the random one
        v0 = orc.verdict(fwd[0].logits, fwd[0].hidden, drafts[0], 30, mode=orc.GREEDY, use_judge=False, top_k=2)
        v1 = orc.verdict(fwd[0].logits, fwd[0].hidden, drafts[0], 30, mode=orc.GREEDY, use_judge=False, top_k=1)
        assert v0.accepted_len == 4 and v1.accepted_len == 1
    finally:
        case.close()


def _target_and_cache(shape, dtype, seed, n_seqs, room=128):
    b = _binding()
    model = helpers.HostModel(shape, dtype, "cpu", seed)
    top = {k: v.cuda() for k, v in model.top.items()}
    layers = [{k: v.cuda() for k, v in lw.items()} for lw in model.layers]
    t = b.Target(shape, top, layers, max_rows=64)
    t.load_judge_head(model.judge_w, 0.0, 0.5)
    return model, t, b.KVCache(t, n_seqs, n_seqs * (room // 16 + 2))


def test_speculative_loop_reproduces_the_targets_greedy_decoding():
    """Draft passes + verification + cache roll-back as a loop.  With the judge off, speculative decoding at
    temperature 0 must emit exactly what the target alone would (Sec. 3.1: the target distribution is kept);
    the first tokens are also checked against the oracle's own greedy continuation."""
    from paper_2510_02329_b200 import loop
    shape, gamma, n_out = synth.TINY, 4, 14
    tm, target, target_kv = _target_and_cache(shape, torch.float32, 0, 2)
    _, draft, draft_kv = _target_and_cache(shape, torch.float32, 1, 2)        # another random model of the same shape
    _, solo, solo_kv = _target_and_cache(shape, torch.float32, 0, 2)
    try:
        prompts = [list(synth.token_ids(shape.vocab, 9, seed=41, stream=3)), list(synth.token_ids(shape.vocab, 5, seed=42, stream=3))]
        dec = loop.SpeculativeDecoder(draft, draft_kv, target, target_kv, [0, 1], gamma)
        dec.prefill(prompts)
        got = dec.generate(n_out, use_judge=False)
        want = [loop.greedy_decode(solo, solo_kv, s, prompts[s], n_out) for s in (0, 1)]
        assert got == want
        assert 0.0 <= dec.mean_accepted_length < gamma       # an unrelated draft is mostly rejected
        # oracle: greedy continuation by full recomputes (tiny model)
        osh, top64 = helpers.oracle_shape(shape), tm.top64()
        seq = list(prompts[0])
        for k in range(4):
            bf, _ = orc.prefill(osh, top64, tm.layer64, np.asarray(seq))
            row = bf.logits[-1]
            srt = np.sort(row)
            if srt[-1] - srt[-2] < 1e-3:
                break
            assert got[0][k] == int(np.argmax(row))
            seq.append(got[0][k])
        # with the judge threshold at 0 every draft is accepted: the loop then follows the draft model
        dec2 = loop.SpeculativeDecoder(draft, draft_kv, target, target_kv, [0, 1], gamma)
        target_kv.rollback([0, 1], [0, 0]); draft_kv.rollback([0, 1], [0, 0])
        dec2.prefill(prompts)
        dec2.generate(10, use_judge=True, theta=0.0)
        assert dec2.mean_accepted_length == gamma
    finally:
        for kv in (target_kv, draft_kv, solo_kv):
            kv.close()
        for t in (target, draft, solo):
            t.close()


def test_speculative_loop_with_the_target_as_its_own_draft_accepts_everything():
    from paper_2510_02329_b200 import loop
    shape, gamma = GQA, 5
    _, target, target_kv = _target_and_cache(shape, torch.bfloat16, 0, 1)
    _, draft, draft_kv = _target_and_cache(shape, torch.bfloat16, 0, 1)
    try:
        prompt = list(synth.token_ids(shape.vocab, 20, seed=43, stream=3))
        dec = loop.SpeculativeDecoder(draft, draft_kv, target, target_kv, [0], gamma)
        dec.prefill([prompt])
        out = dec.generate(24, use_judge=False)
        # a draft pass sees one row, the verification gamma + 1: same model, slightly different rounding, so a
        # rejection can only happen at a near-tie of the two best logits
        assert dec.mean_accepted_length >= gamma - 1.0
        assert len(out[0]) == 24
    finally:
        target_kv.close(); draft_kv.close(); target.close(); draft.close()
