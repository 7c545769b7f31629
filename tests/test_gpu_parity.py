"""GPU parity: the CUDA library through its C ABI against the CPU oracle on the same seeded bytes."""
import numpy as np
import pytest
import torch

import harness
import helpers
from oracle import sj_oracle as orc
from paper_2510_02329_b200 import synth

pytestmark = pytest.mark.gpu

GQA = synth.ModelShape("gqa-small", 3, 256, 4, 2, 64, 512, 1024, rope_theta=5e5)
GQA128 = synth.ModelShape("gqa-hd128", 2, 512, 8, 2, 128, 1024, 2048, rope_theta=5e5, qkv_bias=True)


def _binding():
    from paper_2510_02329_b200 import binding
    return binding


# ------------------------------------------------------------------------------------------------
# kernel level: the skinny GEMM
# ------------------------------------------------------------------------------------------------
GEMM_SHAPES = [(5, 384, 256), (9, 1000, 512), (17, 4096, 4096), (72, 2048, 1024), (1, 128, 64), (16, 256, 8192)]


@pytest.mark.parametrize("R,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("dtype,impl", [(torch.float32, 0), (torch.bfloat16, 0), (torch.bfloat16, 1)],
                         ids=["f32-cudacore", "bf16-cudacore", "bf16-tcgen05"])
def test_gemm_skinny_matches_fp64_matmul(R, N, K, dtype, impl):
    b = _binding()
    a = synth.normal(synth.tensor_key(1, 50, R), (R, K), 1.0, dtype)
    w = synth.normal(synth.tensor_key(1, 51, N), (N, K), 0.02, dtype)
    y = b.gemm_skinny(a.cuda(), w.cuda(), impl).cpu().numpy()
    a64, w64 = helpers.np64(a), helpers.np64(w)
    ref = a64 @ w64.T
    bound = 1e-5 * (np.abs(a64) @ np.abs(w64).T) + 1e-7
    err = np.abs(y - ref)
    assert (err <= bound).all(), f"max err {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}"


@pytest.mark.parametrize("R", [288, 512])
def test_gemm_skinny_tcgen05_many_rows(R):
    b = _binding()
    N, K = 640, 1024
    a = synth.normal(synth.tensor_key(2, 50, R), (R, K), 1.0, torch.bfloat16)
    w = synth.normal(synth.tensor_key(2, 51, N), (N, K), 0.02, torch.bfloat16)
    y = b.gemm_skinny(a.cuda(), w.cuda(), 1).cpu().numpy()
    a64, w64 = helpers.np64(a), helpers.np64(w)
    assert (np.abs(y - a64 @ w64.T) <= 1e-5 * (np.abs(a64) @ np.abs(w64).T) + 1e-7).all()


# ------------------------------------------------------------------------------------------------
# whole step
# ------------------------------------------------------------------------------------------------
def _run(case, mode, temperature=1.0, theta=0.5, use_align=True, use_judge=True, options=None):
    for k, v in (options or {}).items():
        case.target.set_option(k, v)
    v, f = case.run_oracle(mode, temperature, theta, use_align, use_judge)
    g = case.run_gpu(mode, temperature, theta, use_align, use_judge)
    return harness.compare(case, v, f, g, mode, temperature, theta), g


CFG1_VARIANTS = [
    ("f32", torch.float32, {}),
    ("f32-nograph-nopdl", torch.float32, {"graph": 0, "pdl": 0}),
    ("bf16-cudacore", torch.bfloat16, {"gemm_impl": 0}),
    ("bf16-persistent", torch.bfloat16, {"gemm_impl": 1, "step_impl": 1}),
    ("bf16-tcgen05", torch.bfloat16, {"gemm_impl": 1, "step_impl": 0}),
    ("bf16-tcgen05-simt-attn", torch.bfloat16, {"gemm_impl": 1, "step_impl": 0, "attn_impl": 0}),
    ("bf16-tcgen05-nograph", torch.bfloat16, {"gemm_impl": 1, "step_impl": 0, "graph": 0, "pdl": 0}),
]


@pytest.mark.parametrize("name,dtype,options", CFG1_VARIANTS, ids=[v[0] for v in CFG1_VARIANTS])
def test_config1_tiny_target(name, dtype, options):
    """2 layers, d 256, 4 MHA heads of 64, FFN 1024, vocab 4096; batch 1, 128 cached tokens, gamma 4."""
    case = harness.Case(synth.TINY, dtype, [128], 4, seed=0).gpu_setup()
    try:
        exact = 0
        for mode, T in [(orc.GREEDY, 1.0), (orc.SAMPLING, 1.0), (orc.SAMPLING, 0.1)]:
            rep, _ = _run(case, mode, T, options=options)
            exact += rep.exact
            print(name, "mode", mode, "T", T, rep)
        if dtype == torch.float32:
            assert exact >= 2  # fp32 decisions are crisp except true near-ties
    finally:
        case.close()


@pytest.mark.parametrize("dtype,options", [(torch.float32, {}), (torch.bfloat16, {"gemm_impl": 0}),
                                            (torch.bfloat16, {"gemm_impl": 1, "step_impl": 0}),
                                            (torch.bfloat16, {"gemm_impl": 1, "step_impl": 1})],
                         ids=["f32", "bf16-cudacore", "bf16-tcgen05", "bf16-persistent"])
@pytest.mark.parametrize("kv_lens,gamma", [([5, 37, 130], 3), ([15, 16, 17, 0], 5), ([200], 1), ([63, 64], 16)])
def test_ragged_batches_and_page_edges(dtype, options, kv_lens, gamma):
    case = harness.Case(GQA, dtype, kv_lens, gamma, seed=3).gpu_setup()
    try:
        for mode, T in [(orc.GREEDY, 1.0), (orc.SAMPLING, 0.2)]:
            rep, _ = _run(case, mode, T, options=options)
            assert rep.exact + rep.margin == len(kv_lens)
    finally:
        case.close()


@pytest.mark.parametrize("options", [{"gemm_impl": 0}, {"gemm_impl": 1, "step_impl": 0}, {"gemm_impl": 1, "step_impl": 1},
                                     {"gemm_impl": 1, "step_impl": 0, "attn_impl": 2}],
                         ids=["cudacore", "tcgen05", "persistent", "tcgen05-attention"])
def test_head_dim_128_with_qkv_bias(options):
    case = harness.Case(GQA128, torch.bfloat16, [70, 300], 8, seed=4).gpu_setup()
    try:
        for mode, T in [(orc.GREEDY, 1.0), (orc.SAMPLING, 0.2)]:
            _run(case, mode, T, options=options)
    finally:
        case.close()


def test_drafts_following_the_target_are_accepted_and_judge_flags():
    """Drafts that equal the oracle's greedy chain are accepted; ablation flags and theta limits."""
    shape, L, gamma = GQA, 40, 6
    probe = harness.Case(shape, torch.float32, [L], gamma, seed=7)
    # greedy chain from the oracle: feed pending, take argmax, append, repeat
    osh, top = probe.osh, probe.top64
    caches = [[(helpers.np64(k), helpers.np64(v)) for k, v in probe.cache_t[0]]]
    chain, toks = [], [int(probe.inputs.pending[0])]
    for _ in range(gamma - 2):
        fwd = orc.forward_blocks(osh, top, probe.model.layer64, [np.array(toks)], caches)[0]
        chain.append(int(np.argmax(fwd.logits[-1])))
        toks.append(chain[-1])
    drafts = probe.inputs.draft_ids.copy()
    drafts[0, :gamma - 2] = chain
    case = harness.Case(shape, torch.float32, [L], gamma, seed=7, draft_ids=drafts).gpu_setup()
    try:
        rep, g = _run(case, orc.GREEDY, use_judge=False)
        assert rep.exact == 1 and g["accepted_len"][0] >= gamma - 2
        n_off = int(g["accepted_len"][0])
        rep, g = _run(case, orc.GREEDY, theta=0.0)
        assert g["accepted_len"][0] == gamma                         # sigmoid > 0 always
        rep, g = _run(case, orc.GREEDY, theta=1.0)
        assert g["accepted_len"][0] == n_off                         # judge can never fire
        prev = gamma
        for th in (0.3, 0.5, 0.7):
            rep, g = _run(case, orc.GREEDY, theta=th)
            assert rep.exact == 1 and g["accepted_len"][0] <= prev
            prev = int(g["accepted_len"][0])
        rep, g = _run(case, orc.GREEDY, use_align=False)              # judge only
        assert rep.exact == 1
    finally:
        case.close()


def test_commit_second_step_and_rollback():
    b = _binding()
    shape, L, gamma = GQA, 21, 4
    case = harness.Case(shape, torch.float32, [L], gamma, seed=11).gpu_setup()
    try:
        v1, f1 = case.run_oracle(orc.GREEDY, use_judge=True, theta=0.5)
        g1 = case.run_gpu(orc.GREEDY, theta=0.5, commit=True)
        rep = harness.compare(case, v1, f1, g1, orc.GREEDY)
        assert rep.exact == 1
        n = v1[0].accepted_len
        assert case.kv.lengths([0]) == [L + 1 + n]
        # committed cache rows equal the oracle's new rows (first 1+n)
        for l in range(shape.n_layers):
            k, v = case.kv.read(0, l, L, 1 + n)
            assert np.abs(k.cpu().double().numpy() - f1[0].k_new[l][:1 + n]).max() < 1e-4
            assert np.abs(v.cpu().double().numpy() - f1[0].v_new[l][:1 + n]).max() < 1e-4
        # second step: pending is the first step's next token (set on the device by the commit)
        si2 = synth.step_inputs(shape.vocab, 1, gamma, seed=12)
        caches2 = [[(np.concatenate([helpers.np64(case.cache_t[0][l][0]), f1[0].k_new[l][:1 + n]]),
                     np.concatenate([helpers.np64(case.cache_t[0][l][1]), f1[0].v_new[l][:1 + n]]))
                    for l in range(shape.n_layers)]]
        v2, f2 = orc.verify(case.osh, case.top64, case.model.layer64, [v1[0].next_token], si2.draft_ids, caches2,
                            mode=orc.GREEDY, judge_w=case.judge_w64, theta=0.5)
        out = b.VerifyBuffers(1, gamma, shape.d_model, shape.vocab, debug=True)
        b.verify(case.target, case.kv, [0], torch.from_numpy(si2.draft_ids).cuda(), out, commit=False)
        case.target.sync()
        assert np.abs(out.dbg_logits.cpu().numpy()[0] - f2[0].logits).max() < 1e-3
        assert int(out.accepted_len[0]) == v2[0].accepted_len and int(out.next_token[0]) == v2[0].next_token
        # rollback to L and run the first step again: identical outputs
        case.kv.rollback([0], [L])
        g3 = case.run_gpu(orc.GREEDY, theta=0.5, commit=False)
        for key in ("accepted_len", "next_token", "new_kv_len"):
            assert np.array_equal(g1[key], g3[key])
        assert np.array_equal(g1["logits"], g3["logits"])            # bit-reproducible
        # rollback beyond the live length: refused by the host, or flagged by the device
        with pytest.raises(b.SjError) as ei:
            case.kv.rollback([0], [L + 100])
        assert ei.value.status == 3
    finally:
        case.close()


def test_bf16_commit_then_second_step():
    """bf16 model: within a step the library reads the block's own key / value rows from an fp16 copy, later
    steps read the bf16 rows in the pages.  The second step must match an oracle whose cache holds the first
    step's committed rows as the library stored them (rounded to bf16)."""
    b = _binding()
    shape, L, gamma = GQA, 37, 5
    case = harness.Case(shape, torch.bfloat16, [L], gamma, seed=13).gpu_setup()
    try:
        # drafts that follow the target, so that several rows are committed
        case.follow_target(0.9)
        v1, f1 = case.run_oracle(orc.GREEDY, theta=0.5)
        g1 = case.run_gpu(orc.GREEDY, theta=0.5, commit=True)
        rep = harness.compare(case, v1, f1, g1, orc.GREEDY)
        assert rep.exact + rep.margin == 1
        n = int(g1["accepted_len"][0])
        assert case.kv.lengths([0]) == [L + 1 + n]
        caches2 = []
        for l in range(shape.n_layers):
            k, v = case.kv.read(0, l, L, 1 + n)       # committed rows, bf16 as stored
            assert np.abs(k.cpu().double().numpy() - f1[0].k_new[l][:1 + n]).max() < 2e-2
            assert np.abs(v.cpu().double().numpy() - f1[0].v_new[l][:1 + n]).max() < 2e-2
            caches2.append((np.concatenate([helpers.np64(case.cache_t[0][l][0]), helpers.np64(k)]),
                            np.concatenate([helpers.np64(case.cache_t[0][l][1]), helpers.np64(v)])))
        si2 = synth.step_inputs(shape.vocab, 1, gamma, seed=14)
        v2, f2 = orc.verify(case.osh, case.top64, case.model.layer64, [int(g1["next_token"][0])], si2.draft_ids, [caches2],
                            mode=orc.GREEDY, judge_w=case.judge_w64, theta=0.5)
        out = b.VerifyBuffers(1, gamma, shape.d_model, shape.vocab, debug=True)
        b.verify(case.target, case.kv, [0], torch.from_numpy(si2.draft_ids).cuda(), out, commit=False)
        case.target.sync()
        tol = harness.tol_for(torch.bfloat16)
        err = np.abs(out.dbg_logits.cpu().numpy()[0] - f2[0].logits)
        assert (err <= tol.delta(f2[0].logits)).all(), err.max()
        assert np.abs(out.judge_scores.cpu().numpy()[0] - v2[0].judge).max() <= tol.judge_abs
    finally:
        case.close()


def test_rollback_returns_whole_pages_to_the_pool():
    """Pages past a rolled-back length go back to the pool at once: another sequence can take them without
    anybody asking for lengths in between."""
    b = _binding()
    case = harness.Case(GQA, torch.float32, [100, 4], 4, seed=2).gpu_setup(page_slack=0)   # a pool of 10 pages
    try:
        k = torch.zeros((100, GQA.n_kv_heads, GQA.head_dim), dtype=torch.float32, device="cuda")
        with pytest.raises(b.SjError) as ei:        # sequence 0 holds 7 pages: 7 more for sequence 1 do not fit
            case.kv.fill(1, 0, 4, k, k)
        assert ei.value.status == 4
        case.kv.rollback([0], [4])                  # keeps one page of sequence 0
        for l in range(GQA.n_layers):
            case.kv.fill(1, l, 4, k, k)
        case.target.sync()
    finally:
        case.close()


def test_page_pool_exhaustion_is_reported_before_any_launch():
    b = _binding()
    case = harness.Case(GQA, torch.float32, [30], 4, seed=2).gpu_setup(page_slack=0)
    try:
        # the pool holds pages for 30 + 5 tokens (+1); a long block needs more
        with pytest.raises(b.SjError) as ei:
            for _ in range(40):
                case.run_gpu(orc.GREEDY, commit=True, debug=False)
        assert ei.value.status == 4
        case.target.sync()
    finally:
        case.close()


@pytest.mark.parametrize("kind", [0, 1, 2], ids=["gemm-barrier-wait", "ring-barrier-wait", "grid-barrier-poll"])
def test_a_bounded_wait_that_runs_out_is_reported_and_the_library_keeps_working(kind):
    """A device-side wait on something nobody signals gives up after its poll limit: the kernel returns, the next
    sync reports SJ_ERR_TIMEOUT (once), and the following step still matches the oracle."""
    b = _binding()
    case = harness.Case(synth.TINY, torch.bfloat16, [128], 4, seed=0).gpu_setup()
    try:
        case.target.expire_wait(kind, 3000)
        with pytest.raises(b.SjError) as ei:
            case.target.sync()
        assert ei.value.status == 7 and "wait ran out" in str(ei.value)
        case.target.sync()                      # the status word was cleared by the failed sync
        rep, _ = _run(case, orc.GREEDY)
        assert rep.exact + rep.margin == 1
    finally:
        case.close()


def test_bit_reproducible_across_runs():
    case = harness.Case(synth.TINY, torch.bfloat16, [128], 4, seed=0).gpu_setup()
    try:
        a = case.run_gpu(orc.SAMPLING, 1.0)
        c = case.run_gpu(orc.SAMPLING, 1.0)
        for k in a:
            assert np.array_equal(a[k], c[k]), k
    finally:
        case.close()


# ------------------------------------------------------------------------------------------------
# full-width cuts of the benchmark shapes (all widths, head counts and the vocabulary as configured;
# fewer layers and a short synthetic cache so that the fp64 oracle finishes in seconds)
# ------------------------------------------------------------------------------------------------
WIDTH_CASES = [
    ("llama-1b-cut2", synth.LLAMA_1B.cut(2), [300], 8),            # tied embeddings, head_dim 64, group 4
    ("llama-8b-cut2", synth.LLAMA_8B.cut(2), [210], 8),            # config 3's widths
    ("llama-8b-cut1-g16", synth.LLAMA_8B.cut(1), [77], 16),        # 17 rows: two 16-column accumulator chunks
    ("qwen-32b-cut1-b8", synth.QWEN_32B.cut(1), [40, 97, 16, 130, 64, 33, 250, 5], 8),   # 72 rows, qkv bias, F 27648
]


@pytest.mark.parametrize("name,shape,kv_lens,gamma", WIDTH_CASES, ids=[c[0] for c in WIDTH_CASES])
def test_full_width_cuts_of_the_benchmark_shapes(name, shape, kv_lens, gamma):
    case = harness.Case(shape, torch.bfloat16, kv_lens, gamma, seed=5, cache="fill", gen_device="cuda").gpu_setup(
        max_rows=len(kv_lens) * (gamma + 1))
    try:
        for mode, T in [(orc.GREEDY, 1.0), (orc.SAMPLING, 1.0)]:
            rep, _ = _run(case, mode, T)
            assert rep.exact + rep.margin == len(kv_lens)
            print(name, "mode", mode, rep)
    finally:
        case.close()


# ------------------------------------------------------------------------------------------------
# the benchmark's own sizes: every layer, the full vocabulary, the cache length and gamma of the
# workload, in the launch configuration bench.py times (default options, one persistent-kernel launch
# per step).  The fp64 oracle computes the whole step: one layer's weights at a time are copied from
# the device and widened, so the host holds a few GB; about a minute for the 8B shape.
# ------------------------------------------------------------------------------------------------
FULL_CASES = [
    ("cfg2", "cfg2", (0.5,)),
    ("cfg3", "cfg3", (0.3, 0.5, 0.7)),          # the judge-threshold sweep of config 3
    ("cfg3-g4", "cfg3-g4", (0.5,)),             # 5 rows: the 4-slot instantiation of the persistent kernel
    ("cfg3-g16", "cfg3-g16", (0.5,)),           # 17 rows: two 16-row accumulator chunks
    ("cfg4", "cfg4", (0.5,)),                   # 32 ragged sequences, 288 rows, drafts follow the target w.p. 0.6
    ("cfg5", "cfg5", (0.5,)),                   # 64 layers (two launches), qkv bias, 72 rows
]


@pytest.mark.parametrize("name,key,thetas", FULL_CASES, ids=[c[0] for c in FULL_CASES])
def test_full_size_benchmark_workloads(name, key, thetas):
    wl = synth.WORKLOADS[key]
    kv_lens = [int(x) for x in synth.kv_lengths(wl, 0)]
    case = harness.Case(wl.shape, torch.bfloat16, kv_lens, wl.gamma, seed=0, cache="fill", gen_device="cuda").gpu_setup(
        max_rows=len(kv_lens) * (wl.gamma + 1))
    try:
        if wl.draft_match_prob > 0.0:
            case.follow_target(wl.draft_match_prob)
        fwd = case.oracle_forward()                 # once: the forward does not depend on mode or threshold
        for mode, T in [(orc.GREEDY, 1.0), (orc.SAMPLING, 1.0)]:
            for theta in thetas:
                v = case.oracle_verdicts(fwd, mode, T, theta)
                g = case.run_gpu(mode, T, theta)
                rep = harness.compare(case, v, fwd, g, mode, T, theta)
                assert rep.exact + rep.margin == len(kv_lens)
                print(name, "mode", mode, "theta", theta, "margin positions", rep.margin, "of", rep.sequences,
                      "mean accepted length %.2f" % float(np.mean(g["accepted_len"])), rep)
    finally:
        case.close()


T5_CASES = [
    ("gqa128-ragged", GQA128, [70, 300, 1, 128, 129, 0, 2047], 8),     # tile edges: 1, 128, 129 keys; an empty cache
    ("llama-8b-cut2", synth.LLAMA_8B.cut(2), [210, 4096], 8),          # config 3 / 4 widths: group 4, 36 query rows
    ("llama-8b-cut1-g16", synth.LLAMA_8B.cut(1), [777], 16),           # 68 query rows
    ("qwen-32b-cut1", synth.QWEN_32B.cut(1), [40, 1300, 515], 8),      # group 5, qkv bias
]


@pytest.mark.parametrize("name,shape,kv_lens,gamma", T5_CASES, ids=[c[0] for c in T5_CASES])
def test_tcgen05_attention(name, shape, kv_lens, gamma):
    """The attention of the multi-kernel path on tcgen05 (scores in tensor memory), against the oracle and against
    the mma.sync attention on the same inputs."""
    cache = "prefill" if shape is GQA128 else "fill"
    case = harness.Case(shape, torch.bfloat16, kv_lens, gamma, seed=8, cache=cache,
                        gen_device="cpu" if shape is GQA128 else "cuda").gpu_setup(max_rows=len(kv_lens) * (gamma + 1))
    try:
        for mode, T in [(orc.GREEDY, 1.0), (orc.SAMPLING, 1.0)]:
            rep, g = _run(case, mode, T, options={"gemm_impl": 1, "step_impl": 0, "attn_impl": 2})
            assert rep.exact + rep.margin == len(kv_lens)
            rep1, g1 = _run(case, mode, T, options={"gemm_impl": 1, "step_impl": 0, "attn_impl": 1})
            assert np.abs(g["hidden"] - g1["hidden"]).max() < 5e-3
            print(name, "mode", mode, rep)
    finally:
        case.close()


# at least 49 block rows each: the persistent kernel's ring stages then hold a 32 KiB key or value tile
A5_CASES = [
    ("llama-8b-cut2-b6", synth.LLAMA_8B.cut(2), [4096, 210, 1, 129, 128, 777], 8),       # config 3 widths; 36 query rows
    ("llama-8b-cut1-edges", synth.LLAMA_8B.cut(1), [1, 63, 64, 65, 0, 127, 128, 129, 255, 256, 257, 300], 4),  # tile edges; an empty cache
    ("llama-8b-cut2-g10", synth.LLAMA_8B.cut(2), [3000, 500, 40, 1000, 2000], 10),      # 44 query rows
    ("qwen-32b-cut1-b8", synth.QWEN_32B.cut(1), [40, 1300, 515, 2048, 1, 900, 128, 3000], 8),  # group 5 (45 query rows), qkv bias, 36 KiB stages
]


@pytest.mark.parametrize("name,shape,kv_lens,gamma", A5_CASES, ids=[c[0] for c in A5_CASES])
def test_tcgen05_attention_in_persistent_kernel(name, shape, kv_lens, gamma):
    """The persistent kernel's tcgen05 attention phase (128-key tiles through the shared ring, two issuing threads),
    forced on whatever the cache lengths, against the oracle and against the mma.sync phase on the same inputs."""
    case = harness.Case(shape, torch.bfloat16, kv_lens, gamma, seed=8, cache="fill",
                        gen_device="cuda").gpu_setup(max_rows=len(kv_lens) * (gamma + 1))
    try:
        for mode, T in [(orc.GREEDY, 1.0), (orc.SAMPLING, 1.0)]:
            rep, g = _run(case, mode, T, options={"gemm_impl": 1, "step_impl": 1, "attn_impl": 2, "attn_tcgen05_min_tiles": 0})
            assert rep.exact + rep.margin == len(kv_lens)
            rep1, g1 = _run(case, mode, T, options={"gemm_impl": 1, "step_impl": 1, "attn_impl": 1})
            d = np.abs(g["hidden"] - g1["hidden"]).max()
            assert 0 < d < 5e-3 or max(kv_lens) == 0   # close, and not the same code path
            print(name, "mode", mode, rep, "vs mma.sync", d)
    finally:
        case.close()


def test_more_than_256_rows_keep_both_activation_planes():
    """29 sequences x 9 rows = 261 rows: the two bf16 activation planes no longer fit side by side in tensor
    memory and the lo plane is accumulated into the hi plane's columns."""
    kv_lens = [5 + 7 * b for b in range(29)]
    case = harness.Case(GQA, torch.bfloat16, kv_lens, 8, seed=6).gpu_setup(max_rows=29 * 9)
    try:
        for mode, T in [(orc.GREEDY, 1.0), (orc.SAMPLING, 0.5)]:
            rep, g = _run(case, mode, T)
            assert rep.exact + rep.margin == len(kv_lens)
            # the hidden states are as accurate as with few rows (plain bf16 activations are ~30x worse)
            assert rep.max_hidden_err < 2e-3, rep
    finally:
        case.close()


def test_more_layers_than_one_launch_holds():
    """35 layers of the tiny widths: the persistent kernel runs them as two launches (32 + 3); the second
    one starts from the residual stream and sums of squares the first one left."""
    shape = synth.TINY.cut(35)
    case = harness.Case(shape, torch.bfloat16, [70, 19], 4, seed=3).gpu_setup()
    try:
        for mode in (orc.GREEDY, orc.SAMPLING):
            rep, g = _run(case, mode, options={"gemm_impl": 1, "step_impl": 1})
            assert rep.exact + rep.margin == 2
            rep0, g0 = _run(case, mode, options={"gemm_impl": 1, "step_impl": 0})
            assert np.abs(g["hidden"] - g0["hidden"]).max() < 2e-2
    finally:
        case.close()
