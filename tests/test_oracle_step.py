"""Whole-step pins: committing the accepted prefix and verifying again equals one forward over
the concatenated context; generator determinism."""
import numpy as np
import torch

import helpers
from oracle import sj_oracle as orc
from paper_2510_02329_b200 import synth


def test_commit_then_verify_equals_forward_over_concatenated_context():
    shape = synth.ModelShape("s", 2, 64, 4, 2, 16, 128, 97)
    model = helpers.HostModel(shape, torch.float32)
    osh, top = helpers.oracle_shape(shape), model.top64()
    L, gamma = 11, 4
    prefix = synth.token_ids(shape.vocab, L, seed=1)
    _, cache = orc.prefill(osh, top, model.layer64, prefix)
    si = synth.step_inputs(shape.vocab, 1, gamma, seed=2)
    # make the first two drafts match the target so that something is accepted
    tgt_chain = []
    ctx = list(prefix) + [int(si.pending[0])]
    for _ in range(2):
        full, _ = orc.prefill(osh, top, model.layer64, np.array(ctx))
        tgt_chain.append(int(np.argmax(full.logits[-1])))
        ctx.append(tgt_chain[-1])
    drafts = si.draft_ids.copy()
    drafts[0, :2] = tgt_chain
    v, fwd = orc.verify(osh, top, model.layer64, si.pending, drafts, [cache], mode=orc.GREEDY,
                        judge_w=helpers.np64(model.judge_w), use_judge=False)
    v, fwd = v[0], fwd[0]
    assert v.accepted_len >= 2 and v.new_kv_len == L + 1 + v.accepted_len
    keep = 1 + v.accepted_len
    cache2 = [(np.concatenate([cache[l][0], fwd.k_new[l][:keep]]), np.concatenate([cache[l][1], fwd.v_new[l][:keep]]))
              for l in range(shape.n_layers)]
    si2 = synth.step_inputs(shape.vocab, 1, gamma, seed=3)
    v2, fwd2 = orc.verify(osh, top, model.layer64, [v.next_token], si2.draft_ids, [cache2], mode=orc.GREEDY,
                          use_judge=False)
    ctx_all = np.concatenate([prefix, si.pending, drafts[0, :v.accepted_len], [v.next_token], si2.draft_ids[0]])
    full, _ = orc.prefill(osh, top, model.layer64, ctx_all)
    assert np.abs(fwd2[0].logits - full.logits[-(gamma + 1):]).max() < 1e-10
    # rolling back to L and verifying the same block again is the same computation
    v3, _ = orc.verify(osh, top, model.layer64, si.pending, drafts, [cache], mode=orc.GREEDY, use_judge=False)
    assert (v3[0].accepted_len, v3[0].next_token) == (v.accepted_len, v.next_token)


def test_generator_is_sliceable_and_seeded():
    key = synth.tensor_key(0, synth.K_WQ, 3)
    a = synth.normal(key, (1000,), 0.02, torch.float64)
    b = synth.normal(key, (300,), 0.02, torch.float64, start=200)
    assert torch.equal(a[200:500], b)
    c = synth.normal(synth.tensor_key(0, synth.K_WQ, 4), (1000,), 0.02, torch.float64)
    assert not torch.equal(a, c)
    big = synth.normal(key, (400_000,), 1.0, torch.float64)
    assert abs(big.mean().item()) < 0.01 and abs(big.std().item() - 1.0) < 0.01
    assert abs((big ** 4).mean().item() - 3.0) < 0.1
    q = synth.dirichlet_rows(3, 4096, 0.1, seed=0)
    assert np.allclose(q.sum(axis=1), 1.0, atol=1e-5) and q.min() < 1e-20   # heavy lower tail (fp32 underflow to 0 does occur)
    u = synth.uniforms((1000,), seed=0)
    assert u.min() >= 0 and u.max() < 1
    si = synth.step_inputs(50, 2, 3, seed=9)
    assert np.array_equal(si.draft_q_tok[1, 2], si.draft_q_full[1, 2, si.draft_ids[1, 2]])
