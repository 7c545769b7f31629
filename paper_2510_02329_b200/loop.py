"""Host loop of judge speculative decoding around the library's calls (plumbing only).

One cycle (Sec. 3.1 / 3.2 of the paper): the draft model proposes gamma tokens by gamma single-position
decode steps, the target verifies the block in one step (`sj_verify`: alignment test OR judge score above the
threshold, first rejection, emitted token), both caches are cut back to the accepted prefix.  Every model step
-- the draft's decode steps included -- runs in the library's kernels: a decode step is a verification step
over the block [x_t, dummy] whose dummy draft is rejected outright (both tests off), which commits x_t's
K/V row and makes the model's greedy token the next pending token.

This module only moves token ids between the calls and keeps the two caches in step; it draws no random
numbers and computes nothing of the method itself (temperature 0, the paper's setting).
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding


class SpeculativeDecoder:
    """A draft (target, cache) pair and a verifying (target, cache) pair over the same sequence slots."""

    def __init__(self, draft: binding.Target, draft_kv: binding.KVCache, target: binding.Target,
                 target_kv: binding.KVCache, seq_ids: Sequence[int], gamma: int):
        self.draft, self.draft_kv, self.target, self.target_kv = draft, draft_kv, target, target_kv
        self.seq_ids, self.gamma = [int(s) for s in seq_ids], int(gamma)
        self.B = len(self.seq_ids)
        self.lens = [0] * self.B                      # tokens in both caches (they are kept equal)
        self.pending: List[int] = [0] * self.B        # next token to feed (not yet in the caches)
        self.cycles = 0
        self.accepted_total = 0

    # ---- set-up -------------------------------------------------------------------------------
    def prefill(self, prompts: Sequence[Sequence[int]]) -> None:
        """Both caches receive prompt[:-1]; the last prompt token becomes the pending token."""
        for i, (s, prompt) in enumerate(zip(self.seq_ids, prompts)):
            assert len(prompt) >= 1
            if len(prompt) > 1:
                self.draft_kv.prefill(s, prompt[:-1], want_next=False)
                self.target_kv.prefill(s, prompt[:-1], want_next=False)
            self.lens[i] = len(prompt) - 1
            self.pending[i] = int(prompt[-1])

    # ---- one decode step of a model on a subset of the sequences ------------------------------------
    @staticmethod
    def _decode(target: binding.Target, kv: binding.KVCache, seqs: Sequence[int]) -> torch.Tensor:
        """Feed each sequence's pending token, keep its K/V row, return the greedy next tokens (device [n])."""
        n = len(seqs)
        out = binding.VerifyBuffers(n, 1)
        dummy = torch.zeros((n, 1), dtype=torch.int32, device="cuda")
        binding.verify(target, kv, seqs, dummy, out, mode=binding.MODE_GREEDY, use_align=False, use_judge=False, commit=True)
        return out.next_token

    # ---- one cycle ----------------------------------------------------------------------------------
    def cycle(self, use_judge: bool = True, theta: float = -1.0, top_k: int = 0) -> List[List[int]]:
        """Draft gamma tokens, verify, commit.  Returns, per sequence, the tokens this cycle appended to the
        output: the accepted drafts followed by the token the target emitted."""
        B, gamma = self.B, self.gamma
        self.draft_kv.set_pending(self.seq_ids, self.pending)
        self.target_kv.set_pending(self.seq_ids, self.pending)
        drafts = torch.zeros((B, gamma), dtype=torch.int32, device="cuda")
        for j in range(gamma):                                        # the draft's gamma sequential passes
            nxt = self._decode(self.draft, self.draft_kv, self.seq_ids)
            self.draft.stream.synchronize()
            drafts[:, j] = nxt
        out = binding.VerifyBuffers(B, gamma)
        binding.verify(self.target, self.target_kv, self.seq_ids, drafts, out, mode=binding.MODE_GREEDY,
                       use_align=True, use_judge=use_judge, theta=theta, top_k=top_k, commit=True)
        self.target.sync()
        n_acc = out.accepted_len.cpu().numpy()
        emitted = out.next_token.cpu().numpy()
        d_host = drafts.cpu().numpy()
        produced, full = [], []
        for i in range(B):
            n = int(n_acc[i])
            produced.append([int(t) for t in d_host[i, :n]] + [int(emitted[i])])
            self.lens[i] += 1 + n
            self.pending[i] = int(emitted[i])
            if n == gamma:
                full.append(i)
        # the draft's cache holds x_t, d_1 .. d_{gamma-1}: cut it back to the accepted prefix, or, where every
        # draft was accepted, feed it d_gamma as well
        part = [i for i in range(B) if i not in full]
        if part:
            self.draft_kv.rollback([self.seq_ids[i] for i in part], [self.lens[i] for i in part])
        if full:
            seqs = [self.seq_ids[i] for i in full]
            self.draft_kv.set_pending(seqs, [int(d_host[i, gamma - 1]) for i in full])
            self._decode(self.draft, self.draft_kv, seqs)
        self.cycles += 1
        self.accepted_total += int(n_acc.sum())
        return produced

    def generate(self, n_tokens: int, **kw) -> List[List[int]]:
        """Cycles until every sequence has produced at least n_tokens tokens (then truncated)."""
        outs: List[List[int]] = [[] for _ in range(self.B)]
        while min(len(o) for o in outs) < n_tokens:
            for o, p in zip(outs, self.cycle(**kw)):
                o.extend(p)
        return [o[:n_tokens] for o in outs]

    @property
    def mean_accepted_length(self) -> float:
        """Accepted drafts per sequence per cycle (the paper's m counts the emitted token too: add 1)."""
        return self.accepted_total / max(1, self.cycles * self.B)


def greedy_decode(target: binding.Target, kv: binding.KVCache, seq: int, prompt: Sequence[int], n_tokens: int) -> List[int]:
    """Plain greedy decoding with one model: the sequence the speculative loop must reproduce when only the
    alignment test accepts."""
    if len(prompt) > 1:
        kv.prefill(seq, prompt[:-1], want_next=False)
    kv.set_pending([seq], [int(prompt[-1])])
    out = []
    for _ in range(n_tokens):
        nxt = SpeculativeDecoder._decode(target, kv, [seq])
        target.sync()
        out.append(int(nxt.cpu()[0]))
    return out
