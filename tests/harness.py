"""Parity harness: build one verification case, run the oracle and the CUDA library on the same
bytes, and compare with the margin rules (decisions within the float tolerance are counted, not
failed; everything before the first such position must match exactly)."""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np
import torch

import helpers
from oracle import sj_oracle as orc
from paper_2510_02329_b200 import synth


@dataclasses.dataclass
class Tol:
    abs_: float
    rel: float
    judge_abs: float

    def delta(self, x: np.ndarray) -> np.ndarray:
        return self.abs_ + self.rel * np.abs(x)


def tol_for(dtype: torch.dtype, logit_scale: float = 1.0) -> Tol:
    if dtype == torch.bfloat16:
        return Tol(2e-2, 2e-2, 1e-3)
    return Tol(1e-4 * max(1.0, logit_scale), 1e-4, 1e-4)


class Case:
    """Weights, cache and step inputs of one configuration, on the host and on the device."""

    def __init__(self, shape: synth.ModelShape, dtype: torch.dtype, kv_lens, gamma: int, seed: int = 0,
                 cache: str = "prefill", gen_device: str = "cpu", draft_ids: Optional[np.ndarray] = None):
        self.shape, self.dtype, self.gamma, self.seed = shape, dtype, gamma, seed
        self.kv_lens = [int(x) for x in kv_lens]
        self.B = len(self.kv_lens)
        self.model = helpers.HostModel(shape, dtype, gen_device, seed)
        self.osh = helpers.oracle_shape(shape)
        self.top64 = self.model.top64()
        self.judge_w64 = helpers.np64(self.model.judge_w)
        # cache rows in storage dtype, per sequence per layer: (K [L,Hkv,hd], V)
        self.cache_t: List[List[tuple]] = []
        if cache == "prefill":
            for b, L in enumerate(self.kv_lens):
                prefix = synth.token_ids(shape.vocab, L, seed, stream=100 + b)
                _, c = orc.prefill(self.osh, self.top64, self.model.layer64, prefix)
                self.cache_t.append([(helpers.round_to(k, dtype), helpers.round_to(v, dtype)) for k, v in c])
        else:
            for b, L in enumerate(self.kv_lens):
                self.cache_t.append([synth.cache_fill(shape, l, b, L, dtype, gen_device, seed) for l in range(shape.n_layers)])
        self.inputs = synth.step_inputs(shape.vocab, self.B, gamma, seed, draft_ids=draft_ids)

    # ---------------- oracle ----------------
    def _oracle_caches(self):
        """Per sequence, a sequence-like object whose item l is layer l's (K, V) widened to fp64 on demand: the
        cache of a large workload does not fit host memory as fp64 all at once."""
        cache_t = self.cache_t

        class _Layers:
            def __init__(self, seq):
                self.seq = seq

            def __len__(self):
                return len(self.seq)

            def __getitem__(self, l):
                k, v = self.seq[l]
                return helpers.np64(k), helpers.np64(v)

        return [_Layers(seq) for seq in cache_t]

    def oracle_forward(self):
        """The target forward of the step (Eq. 2) for every sequence: independent of mode, temperature and theta."""
        si = self.inputs
        tokens = [np.concatenate([[int(si.pending[b])], np.asarray(si.draft_ids[b], np.int64)]) for b in range(self.B)]
        return orc.forward_blocks(self.osh, self.top64, self.model.layer64, tokens, self._oracle_caches())

    def oracle_verdicts(self, fwd, mode: int, temperature: float = 1.0, theta: float = 0.5, use_align=True, use_judge=True):
        """The acceptance decisions (Eq. 3, Eq. 5, Sec. 3.1-3.2) for a forward computed by oracle_forward()."""
        si = self.inputs
        return [orc.verdict(bf.logits, bf.hidden, np.asarray(si.draft_ids[b]), self.kv_lens[b], mode=mode,
                            temperature=temperature, q_tok=si.draft_q_tok[b], q_full=si.draft_q_full[b],
                            uniforms=si.uniforms[b], judge_w=self.judge_w64, judge_b=0.0, theta=theta,
                            use_align=use_align, use_judge=use_judge) for b, bf in enumerate(fwd)]

    def run_oracle(self, mode: int, temperature: float = 1.0, theta: float = 0.5, use_align=True, use_judge=True):
        si = self.inputs
        return orc.verify(self.osh, self.top64, self.model.layer64, si.pending, si.draft_ids, self._oracle_caches(),
                          mode=mode, temperature=temperature, q_tok=si.draft_q_tok, q_full=si.draft_q_full,
                          uniforms=si.uniforms, judge_w=self.judge_w64, judge_b=0.0, theta=theta, use_align=use_align,
                          use_judge=use_judge)

    # ---------------- CUDA library ----------------
    def gpu_setup(self, max_rows: Optional[int] = None, page_slack: int = 8, shuffle_pages: bool = True):
        from paper_2510_02329_b200 import binding
        dev = "cuda"
        top = {k: v.to(dev) for k, v in self.model.top.items()}
        if self.shape.tied_embeddings:
            top["lm_head"] = top["embed"]
        layers = [{k: v.to(dev) for k, v in lw.items()} for lw in self.model.layers]
        R = self.B * (self.gamma + 1)
        self.target = binding.Target(self.shape, top, layers, max_rows=max_rows or max(R, 8))
        self.target.load_judge_head(self.model.judge_w, 0.0, 0.5)
        pages = sum((L + self.gamma + 1 + 15) // 16 + 1 for L in self.kv_lens) + page_slack
        self.kv = binding.KVCache(self.target, self.B, pages)
        self.seq_ids = list(range(self.B))
        # interleave the fills of different sequences so that their pages are not contiguous
        order = [(b, l) for l in range(self.shape.n_layers) for b in range(self.B)]
        if shuffle_pages:
            step = 48
            maxL = max(self.kv_lens)
            for start in range(0, maxL, step):
                for b in range(self.B):
                    n = min(step, self.kv_lens[b] - start)
                    if n > 0:
                        for l in range(self.shape.n_layers):
                            k, v = self.cache_t[b][l]
                            self.kv.fill(b, l, start, k[start:start + n].to(dev).contiguous(), v[start:start + n].to(dev).contiguous())
        else:
            for b, l in order:
                k, v = self.cache_t[b][l]
                if k.shape[0]:
                    self.kv.fill(b, l, 0, k.to(dev).contiguous(), v.to(dev).contiguous())
        self.kv.set_len(self.seq_ids, self.kv_lens)
        si = self.inputs
        self.d_draft = torch.from_numpy(si.draft_ids).to(dev)
        self.d_qtok = torch.from_numpy(si.draft_q_tok).to(dev)
        self.d_qfull = torch.from_numpy(si.draft_q_full).to(dev)
        self.d_unif = torch.from_numpy(si.uniforms).to(dev)
        return self

    def follow_target(self, match_prob: float):
        """Replace the drafts by ones that follow the target's greedy chain with probability ``match_prob`` per
        position (the chain is read off the library; the drafts are then fixed inputs of both sides)."""
        from paper_2510_02329_b200 import workload
        d = workload.target_following_drafts(self.target, self.kv, self.seq_ids, self.inputs.pending, self.shape.vocab,
                                             self.gamma, match_prob, self.seed)
        self.inputs = synth.step_inputs(self.shape.vocab, self.B, self.gamma, self.seed, draft_ids=d)
        si = self.inputs
        self.d_draft = torch.from_numpy(si.draft_ids).cuda()
        self.d_qtok = torch.from_numpy(si.draft_q_tok).cuda()
        return self

    def run_gpu(self, mode: int, temperature: float = 1.0, theta: float = -1.0, use_align=True, use_judge=True,
                commit: bool = False, debug: bool = True) -> Dict[str, np.ndarray]:
        from paper_2510_02329_b200 import binding
        self.kv.set_pending(self.seq_ids, self.inputs.pending)
        out = binding.VerifyBuffers(self.B, self.gamma, self.shape.d_model, self.shape.vocab, debug=debug)
        binding.verify(self.target, self.kv, self.seq_ids, self.d_draft, out, mode=mode, temperature=temperature,
                       draft_q_tok=self.d_qtok, draft_q_full=self.d_qfull, uniforms=self.d_unif, use_align=use_align,
                       use_judge=use_judge, theta=theta, commit=commit)
        self.target.sync()
        res = {k: getattr(out, k).cpu().numpy() for k in ("accepted_len", "next_token", "judge_scores", "p_draft", "new_kv_len")}
        if debug:
            res["hidden"] = out.dbg_hidden.cpu().numpy()
            res["logits"] = out.dbg_logits.cpu().numpy()
        return res

    def close(self):
        self.kv.close()
        self.target.close()


@dataclasses.dataclass
class Report:
    sequences: int = 0
    exact: int = 0
    margin: int = 0
    max_logit_err: float = 0.0
    max_hidden_err: float = 0.0
    max_judge_err: float = 0.0
    notes: List[str] = dataclasses.field(default_factory=list)


def compare(case: Case, verdicts, fwd, gpu: Dict[str, np.ndarray], mode: int, temperature: float = 1.0,
            theta: float = 0.5, check_float: bool = True) -> Report:
    """Element-wise float comparison and integer comparison under the margin rules."""
    rep = Report()
    gamma = case.gamma
    scale = max(float(np.abs(f.logits).max()) for f in fwd)
    tol = tol_for(case.dtype, scale)
    for b, (v, f) in enumerate(zip(verdicts, fwd)):
        rep.sequences += 1
        if check_float and "logits" in gpu:
            err = np.abs(gpu["logits"][b] - f.logits)
            bound = tol.delta(f.logits)
            rep.max_logit_err = max(rep.max_logit_err, float(err.max()))
            assert (err <= bound).all(), f"seq {b}: logits off by {err.max():.3e} (bound {bound.min():.3e})"
            errh = np.abs(gpu["hidden"][b] - f.hidden)
            rep.max_hidden_err = max(rep.max_hidden_err, float(errh.max()))
            assert (errh <= tol.delta(f.hidden)).all(), f"seq {b}: hidden off by {errh.max():.3e}"
        errj = np.abs(gpu["judge_scores"][b] - v.judge)
        rep.max_judge_err = max(rep.max_judge_err, float(errj.max()))
        assert (errj <= tol.judge_abs).all(), f"seq {b}: judge scores off by {errj.max():.3e}"
        # p(d_j): relative tolerance implied by the logit tolerance (softmax of z/T)
        dz = (tol.abs_ + tol.rel * scale) / temperature
        eps = math.expm1(2 * dz)
        assert np.all(np.abs(gpu["p_draft"][b] - v.p_draft) <= eps * np.maximum(v.p_draft, 1e-30) + 1e-30), \
            f"seq {b}: p_draft {gpu['p_draft'][b]} vs {v.p_draft}"
        # integers
        n_g, n_o = int(gpu["accepted_len"][b]), v.accepted_len
        t_g, t_o = int(gpu["next_token"][b]), v.next_token
        si = case.inputs
        if n_g != n_o:
            j = min(n_g, n_o) + 1                       # first drafted position decided differently
            near_judge = abs(v.judge[j - 1] - theta) <= tol.judge_abs
            if mode == orc.GREEDY:
                near_align = v.margins["top_gap"][j - 1] <= 2 * tol.delta(np.abs(f.logits[j - 1]).max())
            else:
                p, uq = v.p_draft[j - 1], float(si.uniforms[b, j - 1]) * float(si.draft_q_tok[b, j - 1])
                near_align = abs(p - uq) <= eps * max(p, uq)
            assert near_judge or near_align, f"seq {b}: accepted_len {n_g} vs oracle {n_o}, position {j} is not a near-tie"
            rep.margin += 1
            rep.notes.append(f"seq {b}: near-tie at position {j}")
            continue
        assert int(gpu["new_kv_len"][b]) == v.new_kv_len
        if t_g != t_o:
            if mode == orc.GREEDY:
                near = v.margins["top_gap"][n_o] <= 2 * tol.delta(np.abs(f.logits[n_o]).max())
                # the GPU's token must be one of the near-maximal ones
                near = near and (f.logits[n_o].max() - f.logits[n_o][t_g]) <= 2 * tol.delta(np.abs(f.logits[n_o]).max())
            else:
                m = v.margins
                slack = eps * float(m["cdf_total"])
                near = (float(m["cdf_target"]) - float(m["cdf_lo"]) <= slack) or (float(m["cdf_hi"]) - float(m["cdf_target"]) <= slack)
            assert near, f"seq {b}: next_token {t_g} vs oracle {t_o} is not a near-tie"
            rep.margin += 1
            rep.notes.append(f"seq {b}: next-token near-tie")
            continue
        rep.exact += 1
    return rep
