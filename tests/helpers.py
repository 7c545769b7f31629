"""Glue shared by the tests: dtype conversion and building oracle inputs from synthetic tensors."""
from __future__ import annotations

import numpy as np
import torch

from oracle import sj_oracle as orc
from paper_2510_02329_b200 import synth


def np64(t: torch.Tensor) -> np.ndarray:
    """Stored values (already rounded to their storage dtype) upcast exactly to fp64."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_shape(s: synth.ModelShape) -> orc.Shape:
    return orc.Shape(s.n_layers, s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ffn, s.vocab,
                     s.rope_theta, s.rms_eps)


class HostModel:
    """Synthetic weights held as torch tensors (storage dtype) with fp64 views for the oracle."""

    def __init__(self, shape: synth.ModelShape, dtype=torch.float32, device="cpu", seed=0):
        self.shape = shape
        self.dtype = dtype
        self.top = synth.top_weights(shape, dtype, device, seed)
        self.layers = [synth.layer_weights(shape, l, dtype, device, seed) for l in range(shape.n_layers)]
        self.judge_w = synth.judge_head(shape, device, seed)

    def top64(self):
        return {k: np64(v) for k, v in self.top.items()}

    def layer64(self, l):
        return {k: np64(v) for k, v in self.layers[l].items()}


def round_to(x: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x)).to(dtype)
