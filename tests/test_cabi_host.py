"""No-GPU checks of the C ABI: the library loads, exports every declared symbol, and rejects bad
arguments on the host before touching a device."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2510_02329_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "sj.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sj_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = _declared()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), f"{n} declared in sj.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_null_and_range_errors_are_reported_without_a_device():
    lib = binding.load()
    h = C.c_void_p()
    assert lib.sj_create_target(None, None, None, C.byref(h)) == 1
    assert b"null" in lib.sj_last_error()
    cfg = binding.ModelConfig(2, 256, 4, 4, 64, 1024, 4096, 1e4, 1e-5, 0, 0, 0, 0)
    w = binding.Weights()
    assert lib.sj_create_target(C.byref(cfg), C.byref(w), None, C.byref(h)) == 1      # null weights
    bad = binding.ModelConfig(2, 256, 4, 4, 48, 1024, 4096, 1e4, 1e-5, 0, 0, 0, 0)
    assert lib.sj_create_target(C.byref(bad), C.byref(w), None, C.byref(h)) == 2      # head_dim 48
    bad = binding.ModelConfig(2, 256, 4, 3, 64, 1024, 4096, 1e4, 1e-5, 0, 0, 0, 0)
    assert lib.sj_create_target(C.byref(bad), C.byref(w), None, C.byref(h)) == 2      # 4 % 3 != 0
    bad = binding.ModelConfig(0, 256, 4, 4, 64, 1024, 4096, 1e4, 1e-5, 0, 0, 0, 0)
    assert lib.sj_create_target(C.byref(bad), C.byref(w), None, C.byref(h)) == 1
    assert lib.sj_verify(None, None, None, None) == 1
    assert lib.sj_rollback_kv(None, None, None, 1) == 1
    assert lib.sj_kv_create(None, 1, 1, 16, C.byref(h)) == 1
    assert lib.sj_load_judge_head(None, None, 0.0, 0.5) == 1
    assert lib.sj_gemm_skinny(1, 1, 0, 128, 64, None, None, None, None) == 1
    assert lib.sj_destroy_target(None) == 0 and lib.sj_kv_destroy(None) == 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device failure mode")
def test_compute_calls_fail_loudly_without_a_device():
    lib = binding.load()
    n = 2
    arr = (C.c_void_p * n)(*[0x1000] * n)
    w = binding.Weights()
    w.embed = w.lm_head = w.final_norm = 0x1000
    for name in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm_attn", "norm_ffn"):
        setattr(w, name, C.cast(arr, C.POINTER(C.c_void_p)))
    cfg = binding.ModelConfig(2, 256, 4, 4, 64, 1024, 4096, 1e4, 1e-5, 0, 0, 0, 0)
    h = C.c_void_p()
    st = lib.sj_create_target(C.byref(cfg), C.byref(w), None, C.byref(h))
    assert st == 6 and not h.value, lib.sj_last_error()          # SJ_ERR_CUDA, never a silent CPU path


def test_every_included_source_is_a_build_dependency():
    """An edit of any file the library is compiled from must trigger a rebuild."""
    from paper_2510_02329_b200 import build as b
    deps = {os.path.basename(d) for d in b.deps()}
    csrc = os.path.join(ROOT, "paper_2510_02329_b200", "csrc")
    seen, todo = set(), ["sj_api.cu"]
    while todo:
        f = todo.pop()
        if f in seen:
            continue
        seen.add(f)
        for inc in re.findall(r'#include\s+"([^"]+)"', open(os.path.join(csrc, f)).read()):
            name = os.path.basename(inc)
            if os.path.exists(os.path.join(csrc, name)):
                todo.append(name)
            assert name in deps, f"{f} includes {inc}, which the build does not watch"
    assert {"sj_api.cu", "sj_mega.cuh", "sj.h"} <= seen | deps
