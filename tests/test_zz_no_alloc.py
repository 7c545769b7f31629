"""The allocation-free skinny GEMM against the allocating one.

``sj_gemm_skinny_noalloc`` serves callers that may not touch the device allocator (an engine that owns
all GPU memory, a stream capture in progress elsewhere in the process, a latency path that cannot take
cudaFree's device-wide sync).  Its split-K partial sums live in a fixed array inside the library, shared
by all calls and never cleared between them, so the check runs two different problems back to back: the
second must not be disturbed by what the first left behind.  The file name sorts last so that a run that
stops at the first failure has already executed every other test.
"""
import numpy as np
import pytest
import torch

import helpers
from paper_2510_02329_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _problem(seed, R, N, K):
    a = synth.normal(synth.tensor_key(seed, 60, R), (R, K), 1.0, torch.bfloat16).cuda()
    w = synth.normal(synth.tensor_key(seed, 61, N), (N, K), 0.02, torch.bfloat16).cuda()
    return a, w


def test_noalloc_gemm_matches_allocating_gemm_on_two_calls_in_a_row():
    # deep split first (K/64 = 64 blocks per tile over all SMs), then a wider, shallower problem whose
    # partial sums overlay the first call's leftovers at different offsets
    problems = [(9, 1024, 4096), (17, 2048, 1024)]
    outs = []
    for seed, (R, N, K) in enumerate(problems):
        a, w = _problem(seed + 5, R, N, K)
        y = torch.full((R, N), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        # The library counts its own cudaMalloc / cudaFree calls (torch's allocator statistics cannot see
        # them: the library never allocates through torch).  Free device memory is compared as well: it
        # would show a leak, though not an allocation that is released again before the call returns.
        calls, free_before = binding.device_memory_calls(), torch.cuda.mem_get_info()[0]
        binding.gemm_skinny_noalloc(a, w, y)
        assert binding.device_memory_calls() == calls, "the allocation-free entry point allocated or freed device memory"
        if seed > 0:    # the first call may load the library's kernels onto the device
            assert torch.cuda.mem_get_info()[0] == free_before
        ref = binding.gemm_skinny(a, w, 1)
        assert binding.device_memory_calls() > calls    # the counter does see the allocating entry point
        torch.cuda.synchronize()
        outs.append((a, w, y.cpu().numpy(), ref.cpu().numpy()))
    for a, w, y, ref in outs:
        a64, w64 = helpers.np64(a), helpers.np64(w)
        bound = 1e-5 * (np.abs(a64) @ np.abs(w64).T) + 1e-7    # the tolerance of the other GEMM tests
        assert np.isfinite(y).all()
        assert (np.abs(y - ref) <= bound).all(), f"max diff {np.abs(y - ref).max():.3e}"
        assert (np.abs(y - a64 @ w64.T) <= bound).all()


def test_noalloc_gemm_refuses_problems_beyond_its_scratch():
    R, N, K = 512, 8192, 64          # 4 * 512 * 8192 bytes of partial sums alone exceed the 8 MiB array
    a = torch.zeros((R, K), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((N, K), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((R, N), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.SjError) as ei:
        binding.gemm_skinny_noalloc(a, w, y)
    assert ei.value.status == 2 and "scratch" in str(ei.value)
