"""Device-side set-up of a benchmark / full-size parity workload: synthetic weights drawn on the
GPU, a synthetic paged KV cache, and seeded step inputs.  Plumbing only (torch for memory)."""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from . import binding, synth


def target_following_drafts(target: "binding.Target", kv: "binding.KVCache", seq_ids, pending, vocab: int, gamma: int,
                            match_prob: float, seed: int = 0) -> np.ndarray:
    """Draft ids ``[B, gamma]`` that equal the target's greedy token, given the block so far, with probability
    ``match_prob`` per position and are uniform over the vocabulary otherwise.

    The greedy token after ``[x_t, d_1 .. d_j]`` is read off the library itself: a step over those j drafts
    with the alignment test off and the judge threshold at 0 accepts every position (a sigmoid is positive),
    so its next token is the arg max of the block's last row.  gamma such steps (uncommitted: the cache is left
    as it was) give the chain position by position; the choices are seeded and the drafts are then fixed inputs.
    """
    B = len(seq_ids)
    rng = np.random.Generator(np.random.Philox(key=[seed, 21]))
    follow = rng.random((B, gamma)) < match_prob
    other = rng.integers(0, vocab, size=(B, gamma), dtype=np.int64).astype(np.int32)
    drafts = np.zeros((B, gamma), dtype=np.int32)
    kv.set_pending(seq_ids, pending)
    for j in range(gamma):
        if j == 0:
            # a one-draft block with both tests off rejects at once: the next token is row 0's arg max
            blk, flags = torch.zeros((B, 1), dtype=torch.int32, device="cuda"), dict(use_align=False, use_judge=False)
        else:
            blk = torch.from_numpy(np.ascontiguousarray(drafts[:, :j])).cuda()
            flags = dict(use_align=False, use_judge=True, theta=0.0)
        out = binding.VerifyBuffers(B, blk.shape[1])
        binding.verify(target, kv, seq_ids, blk, out, mode=binding.MODE_GREEDY, commit=False, **flags)
        target.sync()
        assert j == 0 or bool((out.accepted_len == j).all()), "a judge threshold of 0 must accept every position"
        greedy = out.next_token.cpu().numpy()
        drafts[:, j] = np.where(follow[:, j], greedy, other[:, j])
    return drafts


class DeviceWorkload:
    def __init__(self, wl: synth.Workload, dtype: torch.dtype = torch.bfloat16, seed: int = 0,
                 n_layers: Optional[int] = None, stream: Optional[torch.cuda.Stream] = None,
                 draft_ids: Optional[np.ndarray] = None):
        self.wl = wl
        shape = wl.shape if n_layers is None else wl.shape.cut(n_layers)
        self.shape, self.dtype, self.seed = shape, dtype, seed
        dev = "cuda"
        self.top = synth.top_weights(shape, dtype, dev, seed)
        self.layers = [synth.layer_weights(shape, l, dtype, dev, seed) for l in range(shape.n_layers)]
        self.judge_w = synth.judge_head(shape, dev, seed)
        self.B, self.gamma = wl.batch, wl.gamma
        self.R = self.B * (self.gamma + 1)
        self.target = binding.Target(shape, self.top, self.layers, max_rows=max(self.R, 16), stream=stream)
        self.target.load_judge_head(self.judge_w, 0.0, 0.5)
        self.kv_lens: List[int] = [int(x) for x in synth.kv_lengths(wl, seed)]
        ps = wl.page_size
        pages = sum((L + 2 * (self.gamma + 1) + ps - 1) // ps + 1 for L in self.kv_lens) + 8
        self.kv = binding.KVCache(self.target, self.B, pages, ps)
        self.seq_ids = list(range(self.B))
        # fill round-robin over sequences in 256-token pieces so that a sequence's pages interleave
        # with the others' in the pool (block tables are never contiguous runs)
        piece = 256
        first = [synth.cache_fill(shape, 0, b, L, dtype, dev, seed) for b, L in enumerate(self.kv_lens)]
        for s0 in range(0, max(self.kv_lens), piece):
            for b, L in enumerate(self.kv_lens):
                n = min(piece, L - s0)
                if n > 0:
                    self.kv.fill(b, 0, s0, first[b][0][s0:s0 + n], first[b][1][s0:s0 + n])
        del first
        for l in range(1, shape.n_layers):
            for b, L in enumerate(self.kv_lens):
                k, v = synth.cache_fill(shape, l, b, L, dtype, dev, seed)
                self.kv.fill(b, l, 0, k, v)
        self.kv.set_len(self.seq_ids, self.kv_lens)
        self.inputs = synth.step_inputs(shape.vocab, self.B, self.gamma, seed, draft_ids=draft_ids)
        if draft_ids is None and wl.draft_match_prob > 0.0:
            d = target_following_drafts(self.target, self.kv, self.seq_ids, self.inputs.pending, shape.vocab, self.gamma,
                                        wl.draft_match_prob, seed)
            self.inputs = synth.step_inputs(shape.vocab, self.B, self.gamma, seed, draft_ids=d)
        self.upload_inputs()
        self.out = binding.VerifyBuffers(self.B, self.gamma)
        torch.cuda.synchronize()

    def upload_inputs(self) -> None:
        si = self.inputs
        self.d_draft = torch.from_numpy(si.draft_ids).cuda()
        self.d_qtok = torch.from_numpy(si.draft_q_tok).cuda()
        self.d_qfull = torch.from_numpy(si.draft_q_full).cuda()
        self.d_unif = torch.from_numpy(si.uniforms).cuda()

    def step(self, mode: int = binding.MODE_GREEDY, commit: bool = True, out: Optional[binding.VerifyBuffers] = None,
             **kw) -> None:
        """One verification step from the initial cache state (pending reset, verify, rollback)."""
        self.kv.set_pending(self.seq_ids, self.inputs.pending)
        binding.verify(self.target, self.kv, self.seq_ids, self.d_draft, out or self.out, mode=mode,
                       draft_q_tok=self.d_qtok, draft_q_full=self.d_qfull, uniforms=self.d_unif, commit=commit, **kw)
        if commit:
            self.kv.rollback(self.seq_ids, self.kv_lens)

    # ---- byte / flop accounting (algorithmic: every weight and live cache byte once) ----
    def weight_bytes(self) -> int:
        return self.shape.streamed_params() * self.top["embed"].element_size()

    def kv_bytes(self) -> int:
        return sum(self.kv_lens) * self.shape.kv_bytes_per_token(self.top["embed"].element_size())

    def launches_per_step(self, mode: int = binding.MODE_GREEDY, commit: bool = True) -> int:
        n = 2 + 10 * self.shape.n_layers + 2 + (1 if mode == binding.MODE_SAMPLING else 0)
        return n + (1 if commit else 0)

    def close(self) -> None:
        self.kv.close()
        self.target.close()
