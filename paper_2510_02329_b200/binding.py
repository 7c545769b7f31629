"""Thin ctypes binding of ``include/sj.h``: argument marshalling only.

Every step of the verification path runs inside ``libsjverify.so``; this module turns torch
tensors into raw device pointers and checks return codes.  There is no fallback: if the library
is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import build as _build

SJ_OK = 0
STATUS_NAMES = {0: "SJ_OK", 1: "SJ_ERR_INVALID_ARG", 2: "SJ_ERR_SHAPE", 3: "SJ_ERR_STATE", 4: "SJ_ERR_OOM",
                5: "SJ_ERR_UNSUPPORTED", 6: "SJ_ERR_CUDA", 7: "SJ_ERR_TIMEOUT"}
DTYPE_F32, DTYPE_BF16 = 0, 1
MODE_GREEDY, MODE_SAMPLING = 0, 1

EXPORTS = ["sj_create_target", "sj_destroy_target", "sj_load_judge_head", "sj_set_option", "sj_sync",
           "sj_kv_create", "sj_kv_destroy", "sj_kv_fill", "sj_kv_read", "sj_kv_set_len", "sj_kv_set_pending",
           "sj_kv_len", "sj_verify", "sj_rollback_kv", "sj_gemm_skinny", "sj_gemm_skinny_noalloc", "sj_last_error",
           "sj_kernel_time", "sj_step_trace", "sj_device_memory_calls", "sj_debug_expire_wait", "sj_prefill", "sj_semantic_score"]


class SjError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class ModelConfig(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, C.c_int) for n in ("dtype", "tied_embeddings", "qkv_bias", "max_rows")]


_PP = C.POINTER(C.c_void_p)


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, _PP) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm_attn", "norm_ffn",
                                   "bq", "bk", "bv")]


class VerifyArgs(C.Structure):
    _fields_ = [("B", C.c_int), ("gamma", C.c_int), ("seq_ids", C.POINTER(C.c_int)), ("draft_ids", C.c_void_p),
                ("draft_q_tok", C.c_void_p), ("draft_q_full", C.c_void_p), ("uniforms", C.c_void_p),
                ("mode", C.c_int), ("temperature", C.c_float), ("use_align", C.c_int), ("use_judge", C.c_int),
                ("theta_override", C.c_float), ("commit", C.c_int), ("theta_per_seq", C.POINTER(C.c_float)),
                ("top_k", C.c_int), ("accept_all", C.c_int)]


class VerifyOut(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("accepted_len", "next_token", "judge_scores", "p_draft", "new_kv_len",
                                          "dbg_hidden", "dbg_logits", "logp_draft")]


_lib = None


def load(build_if_needed: bool = True) -> C.CDLL:
    """Load ``libsjverify.so`` (compiling it first when the sources are newer and nvcc is present)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.lib_path()
    if build_if_needed and _build.needs_build():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        if os.path.exists(nvcc):
            _build.build()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2510_02329_b200.build`; there is no fallback path")
    lib = C.CDLL(path)
    lib.sj_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name != "sj_last_error":
            getattr(lib, name).restype = C.c_int
    lib.sj_debug_expire_wait.argtypes = [C.c_void_p, C.c_int, C.c_uint]
    lib.sj_semantic_score.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.c_int,
                                      C.POINTER(C.c_float)]
    lib.sj_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_int)]
    lib.sj_device_memory_calls.restype = C.c_long
    lib.sj_device_memory_calls.argtypes = []
    lib.sj_create_target.argtypes = [C.POINTER(ModelConfig), C.POINTER(Weights), C.c_void_p, C.POINTER(C.c_void_p)]
    lib.sj_destroy_target.argtypes = [C.c_void_p]
    lib.sj_load_judge_head.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.c_float, C.c_float]
    lib.sj_set_option.argtypes = [C.c_void_p, C.c_char_p, C.c_int]
    lib.sj_sync.argtypes = [C.c_void_p]
    lib.sj_kernel_time.argtypes = [C.c_void_p, C.c_char_p, C.POINTER(C.c_double), C.POINTER(C.c_long)]
    lib.sj_kv_create.argtypes = [C.c_void_p, C.c_int, C.c_long, C.c_int, C.POINTER(C.c_void_p)]
    lib.sj_kv_destroy.argtypes = [C.c_void_p]
    lib.sj_kv_fill.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
    lib.sj_kv_read.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
    lib.sj_kv_set_len.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_int]
    lib.sj_kv_set_pending.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_int]
    lib.sj_kv_len.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_int]
    lib.sj_verify.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(VerifyArgs), C.POINTER(VerifyOut)]
    lib.sj_rollback_kv.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_int]
    lib.sj_gemm_skinny.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_void_p]
    lib.sj_step_trace.argtypes = [C.c_void_p, C.POINTER(C.c_ulonglong), C.c_int, C.POINTER(C.c_int)]
    lib.sj_gemm_skinny_noalloc.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    _lib = lib
    return lib


def check(status: int) -> None:
    if status != SJ_OK:
        raise SjError(status, load().sj_last_error().decode("utf-8", "replace"))


def _iarr(xs: Sequence[int]):
    return (C.c_int * len(xs))(*[int(x) for x in xs])


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return t.data_ptr()


def _dtype_code(dt: torch.dtype) -> int:
    return {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[dt]


class Target:
    """``sj_create_target`` + ``sj_load_judge_head``; holds references to the borrowed weights."""

    def __init__(self, shape, top: Dict[str, torch.Tensor], layers: List[Dict[str, torch.Tensor]],
                 max_rows: int = 64, stream: Optional[torch.cuda.Stream] = None):
        lib = load()
        self._lib = lib
        self._keep = (top, layers)
        dt = top["embed"].dtype
        self.dtype = dt
        self.shape = shape
        self.stream = stream if stream is not None else torch.cuda.Stream()
        cfg = ModelConfig(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                          shape.d_ffn, shape.vocab, shape.rope_theta, shape.rms_eps, _dtype_code(dt),
                          int(shape.tied_embeddings), int(shape.qkv_bias), max_rows)
        w = Weights()
        w.embed, w.lm_head, w.final_norm = _ptr(top["embed"]), _ptr(top["lm_head"]), _ptr(top["final_norm"])
        self._arrays = {}
        for name in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm_attn", "norm_ffn", "bq", "bk", "bv"):
            if name in layers[0]:
                arr = (C.c_void_p * len(layers))(*[_ptr(l[name]) for l in layers])
                self._arrays[name] = arr
                setattr(w, name, C.cast(arr, _PP))
        self.handle = C.c_void_p()
        check(lib.sj_create_target(C.byref(cfg), C.byref(w), C.c_void_p(self.stream.cuda_stream), C.byref(self.handle)))

    def load_judge_head(self, w: torch.Tensor, bias: float, theta: float) -> None:
        wh = np.ascontiguousarray(w.detach().float().cpu().numpy())
        check(self._lib.sj_load_judge_head(self.handle, wh.ctypes.data_as(C.POINTER(C.c_float)), bias, theta))

    def set_option(self, name: str, value: int) -> None:
        check(self._lib.sj_set_option(self.handle, name.encode(), int(value)))

    def sync(self) -> None:
        check(self._lib.sj_sync(self.handle))

    def expire_wait(self, kind: int, max_polls: int = 2000) -> None:
        """``sj_debug_expire_wait``: queue a one-block kernel whose bounded wait runs out (a drill for SJ_ERR_TIMEOUT)."""
        check(self._lib.sj_debug_expire_wait(self.handle, int(kind), int(max_polls)))

    def kernel_time(self, name: str):
        """(total ms, launches) of the event-bracketed launches whose name starts with ``name``."""
        ms, n = C.c_double(), C.c_long()
        check(self._lib.sj_kernel_time(self.handle, name.encode(), C.byref(ms), C.byref(n)))
        return ms.value, n.value

    def step_trace(self, max_entries: int = 2048 + 16 * 512 + 2 * 32 * 256):
        """Timeline (ns) of the last persistent-kernel step run with option ``trace`` = 1."""
        buf = (C.c_ulonglong * max_entries)()
        n = C.c_int()
        check(self._lib.sj_step_trace(self.handle, buf, max_entries, C.byref(n)))
        return list(buf[: n.value])

    def close(self) -> None:
        if self.handle:
            self._lib.sj_destroy_target(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class KVCache:
    def __init__(self, target: Target, max_seqs: int, max_pages: int, page_size: int = 16):
        self._lib = target._lib
        self.target = target
        self.handle = C.c_void_p()
        check(self._lib.sj_kv_create(target.handle, max_seqs, max_pages, page_size, C.byref(self.handle)))

    def fill(self, seq: int, layer: int, start: int, k: torch.Tensor, v: torch.Tensor) -> None:
        assert k.dtype == self.target.dtype and v.dtype == self.target.dtype and k.shape == v.shape
        self.target.stream.wait_stream(torch.cuda.current_stream())
        k.record_stream(self.target.stream)
        v.record_stream(self.target.stream)
        check(self._lib.sj_kv_fill(self.handle, seq, layer, start, k.shape[0], _ptr(k), _ptr(v)))

    def read(self, seq: int, layer: int, start: int, n: int):
        s = self.target.shape
        k = torch.empty((n, s.n_kv_heads, s.head_dim), dtype=self.target.dtype, device="cuda")
        v = torch.empty_like(k)
        self.target.stream.wait_stream(torch.cuda.current_stream())
        check(self._lib.sj_kv_read(self.handle, seq, layer, start, n, _ptr(k), _ptr(v)))
        return k, v

    def set_len(self, seq_ids, lens) -> None:
        check(self._lib.sj_kv_set_len(self.handle, _iarr(seq_ids), _iarr(lens), len(seq_ids)))

    def set_pending(self, seq_ids, tokens) -> None:
        check(self._lib.sj_kv_set_pending(self.handle, _iarr(seq_ids), _iarr(tokens), len(seq_ids)))

    def lengths(self, seq_ids) -> List[int]:
        out = (C.c_int * len(seq_ids))()
        check(self._lib.sj_kv_len(self.handle, _iarr(seq_ids), out, len(seq_ids)))
        return list(out)

    def prefill(self, seq: int, tokens, want_next: bool = True) -> Optional[int]:
        """``sj_prefill``: append known tokens to a sequence through the verification kernels; returns the
        target's greedy token after the last one (or None without ``want_next``)."""
        nxt = C.c_int(-1)
        check(self._lib.sj_prefill(self.target.handle, self.handle, int(seq), _iarr(tokens), len(tokens),
                                   C.byref(nxt) if want_next else None))
        return int(nxt.value) if want_next else None

    def semantic_score(self, seq: int, y_i: int, z_i: int, future):
        """``sj_semantic_score``: (s, s_prefix) of replacing y_i by z_i given the sequence's cache, its pending
        token y_{i-1} and the future tokens."""
        out = (C.c_float * 2)()
        check(self._lib.sj_semantic_score(self.target.handle, self.handle, int(seq), int(y_i), int(z_i), _iarr(future),
                                          len(future), out))
        return float(out[0]), float(out[1])

    def rollback(self, seq_ids, new_len) -> None:
        check(self._lib.sj_rollback_kv(self.handle, _iarr(seq_ids), _iarr(new_len), len(seq_ids)))

    def close(self) -> None:
        if self.handle:
            self._lib.sj_kv_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class VerifyBuffers:
    """Device outputs of ``sj_verify`` for a fixed (B, gamma)."""

    def __init__(self, B: int, gamma: int, d_model: int = 0, vocab: int = 0, debug: bool = False):
        dev = "cuda"
        self.accepted_len = torch.zeros(B, dtype=torch.int32, device=dev)
        self.next_token = torch.zeros(B, dtype=torch.int32, device=dev)
        self.judge_scores = torch.zeros(B, gamma, dtype=torch.float32, device=dev)
        self.p_draft = torch.zeros(B, gamma, dtype=torch.float32, device=dev)
        self.new_kv_len = torch.zeros(B, dtype=torch.int32, device=dev)
        self.dbg_hidden = torch.zeros(B, gamma + 1, d_model, dtype=torch.float32, device=dev) if debug else None
        self.dbg_logits = torch.zeros(B, gamma + 1, vocab, dtype=torch.float32, device=dev) if debug else None
        self.logp_draft = torch.zeros(B, gamma, dtype=torch.float32, device=dev)

    def struct(self) -> VerifyOut:
        return VerifyOut(_ptr(self.accepted_len), _ptr(self.next_token), _ptr(self.judge_scores), _ptr(self.p_draft),
                         _ptr(self.new_kv_len), _ptr(self.dbg_hidden), _ptr(self.dbg_logits), _ptr(self.logp_draft))


def verify(target: Target, kv: KVCache, seq_ids: Sequence[int], draft_ids: torch.Tensor, out: VerifyBuffers, *,
           mode: int = MODE_GREEDY, temperature: float = 1.0, draft_q_tok: Optional[torch.Tensor] = None,
           draft_q_full: Optional[torch.Tensor] = None, uniforms: Optional[torch.Tensor] = None,
           use_align: bool = True, use_judge: bool = True, theta: float = -1.0, commit: bool = True,
           theta_per_seq: Optional[Sequence[float]] = None, top_k: int = 0, accept_all: bool = False) -> None:
    """``sj_verify``: asynchronous on the target's stream; results land in ``out``."""
    B, gamma = draft_ids.shape
    assert draft_ids.dtype == torch.int32
    ids = _iarr(seq_ids)
    args = VerifyArgs(B, gamma, ids, _ptr(draft_ids), _ptr(draft_q_tok), _ptr(draft_q_full), _ptr(uniforms), mode,
                      temperature, int(use_align), int(use_judge), theta, int(commit),
                      (C.c_float * B)(*[float(x) for x in theta_per_seq]) if theta_per_seq is not None else None,
                      int(top_k), int(accept_all))
    o = out.struct()
    target.stream.wait_stream(torch.cuda.current_stream())   # inputs were produced on the caller's stream
    check(target._lib.sj_verify(target.handle, kv.handle, C.byref(args), C.byref(o)))


def gemm_skinny(a: torch.Tensor, w: torch.Tensor, impl: int) -> torch.Tensor:
    """``sj_gemm_skinny``: y[R, N] fp32 = a[R, K] . w[N, K]^T."""
    R, K = a.shape
    N = w.shape[0]
    y = torch.empty((R, N), dtype=torch.float32, device=a.device)
    check(load().sj_gemm_skinny(_dtype_code(a.dtype), impl, R, N, K, _ptr(a), _ptr(w), _ptr(y),
                                C.c_void_p(torch.cuda.current_stream().cuda_stream)))
    return y


def gemm_skinny_noalloc(a: torch.Tensor, w: torch.Tensor, y: torch.Tensor) -> None:
    """``sj_gemm_skinny_noalloc``: y[R, N] fp32 = a[R, K] . w[N, K]^T (bf16 inputs) into the caller's ``y``.

    For callers that cannot allocate device memory (their engine owns all of it, a capture is in progress
    on another thread, or a cudaFree-induced device sync is unaffordable): the library's partial-sum
    scratch is a fixed array inside the library image, so this wrapper allocates nothing either.
    """
    R, K = a.shape
    N = w.shape[0]
    assert a.dtype == torch.bfloat16 and w.dtype == torch.bfloat16 and y.dtype == torch.float32 and y.shape == (R, N)
    check(load().sj_gemm_skinny_noalloc(R, N, K, _ptr(a), _ptr(w), _ptr(y),
                                        C.c_void_p(torch.cuda.current_stream().cuda_stream)))


def device_memory_calls() -> int:
    """``sj_device_memory_calls``: cudaMalloc / cudaFree calls the library has made so far in this process."""
    return int(load().sj_device_memory_calls())
