/*
 * sj.h -- C ABI of the B200 (sm_100a) verification step for judge speculative decoding.
 *
 * One call, sj_verify(), runs the target decoder over the block [x_t, d_1 .. d_gamma] of each
 * sequence against a paged KV cache (Eq. 2), forms the target probabilities p and the final
 * hidden states h (Eq. 4), applies the probability-ratio acceptance test (Eq. 3; at
 * temperature 0 the strict "draft == target greedy token" test of Sec. 3.1), the judge
 * verifier  Verifier(h) = sigmoid(w.h + b) > theta  (Eq. 5), accepts a token if EITHER test
 * passes (Sec. 3.2, App. D.2), stops at the first rejection (Sec. 3.1), emits the next token
 * and sets the cache length.  Every step runs in hand-written CUDA kernels; there is no CPU
 * fallback: without a CUDA device every compute call returns SJ_ERR_CUDA.
 *
 * Conventions
 *   - All matrices are row-major [out_features, in_features] (y = W x), dtype = config.dtype.
 *   - "device" pointers are CUDA device pointers on the device current at sj_create_target();
 *     "host" pointers are ordinary host memory.  The caller owns every buffer it passes in.
 *     Weights are BORROWED: they must stay valid and unchanged for the life of the handle.
 *   - The library owns its handles, the KV page pool and its workspace (cudaMalloc'ed at
 *     creation / first use, freed by the destroy calls).
 *   - Every call returns an sj_status; sj_last_error() gives a message for the calling thread.
 *     Argument errors are detected on the host before any launch.  sj_verify() and
 *     sj_rollback_kv() are asynchronous on the target's stream; errors only the device can see
 *     (a bounded wait that ran out, a rollback beyond the true length) are recorded in a device
 *     status word and returned by the next sj_sync().
 *   - One stream per target; calls on one handle are not re-entrant.
 *   - Row j (0..gamma) of a sequence's block: row 0's input is the pending token x_t (set by
 *     sj_kv_set_pending() or by the previous committed sj_verify()), row j>=1's input is d_j.
 *     Row j sits at absolute position kv_len + j.  Row j's logits are the target distribution for
 *     drafted position j+1 (row gamma: the bonus token); row j's final hidden state is the judge
 *     input for d_j.
 */
#ifndef SJ_H_
#define SJ_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SJ_OK = 0,
  SJ_ERR_INVALID_ARG = 1, /* null pointer, value out of range */
  SJ_ERR_SHAPE = 2,       /* dimensions the kernels do not support */
  SJ_ERR_STATE = 3,       /* call not valid in the handle's current state */
  SJ_ERR_OOM = 4,         /* page pool or device memory exhausted (nothing was launched) */
  SJ_ERR_UNSUPPORTED = 5,
  SJ_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed (includes "no device") */
  SJ_ERR_TIMEOUT = 7      /* a bounded device-side wait ran out */
} sj_status;

typedef struct sj_target sj_target; /* config + borrowed weights + judge head + workspace */
typedef struct sj_kv sj_kv;         /* page pool, block tables, kv_len[], pending[] */

enum { SJ_DTYPE_F32 = 0, SJ_DTYPE_BF16 = 1 };
enum { SJ_MODE_GREEDY = 0, SJ_MODE_SAMPLING = 1 };

enum {
  SJ_MAX_BATCH = 256,  /* sequences per sj_verify() call */
  SJ_MAX_GAMMA = 31,   /* drafted tokens per sequence */
  SJ_MAX_ROWS = 512    /* B * (gamma + 1) */
};

/* Decoder shape.  Pre-norm decoder: RMSNorm, rotary embedding (rotate-half pairing, angle
 * pos * rope_theta^(-2i/head_dim)), grouped-query attention, SwiGLU FFN -- the Llama-3 /
 * Qwen-2.5 family the paper evaluates (Sec. 4).  max_rows sizes the workspace: the largest
 * B*(gamma+1) any sj_verify() call will use (0 -> 64). */
typedef struct {
  int n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rope_theta, rms_eps;
  int dtype;            /* SJ_DTYPE_*: storage type of weights, activations and the KV cache */
  int tied_embeddings;  /* informational; pass the same pointer for embed and lm_head */
  int qkv_bias;         /* 1: bq/bk/bv are read */
  int max_rows;
} sj_model_config;

/* Device pointers to the weights; the per-layer members are HOST arrays of n_layers device
 * pointers (the arrays themselves are copied, the tensors are borrowed).
 *   embed, lm_head [vocab, d_model]; final_norm, norm_attn[l], norm_ffn[l] [d_model];
 *   wq [Hq*hd, d]; wk, wv [Hkv*hd, d]; wo [d, Hq*hd]; w_gate, w_up [d_ffn, d]; w_down [d, d_ffn];
 *   bq [Hq*hd]; bk, bv [Hkv*hd] (may be NULL when qkv_bias == 0).
 * bf16 matrices must be 16-byte aligned. */
typedef struct {
  const void *embed, *lm_head, *final_norm;
  const void *const *wq, *const *wk, *const *wv, *const *wo, *const *w_gate, *const *w_up, *const *w_down;
  const void *const *norm_attn, *const *norm_ffn;
  const void *const *bq, *const *bk, *const *bv;
} sj_weights;

/* Create a target on the current CUDA device.  cuda_stream is a cudaStream_t (NULL: the legacy
 * default stream) on which all work of this handle and of its KV objects is issued.
 * Errors: INVALID_ARG (null / non-positive dims), SHAPE (head_dim not in {64,128}, odd group,
 * dims not multiples of 8 ...), CUDA, OOM. */
sj_status sj_create_target(const sj_model_config *cfg, const sj_weights *w, void *cuda_stream, sj_target **out);
sj_status sj_destroy_target(sj_target *t);

/* Judge verifier head of Eq. 5: score = sigmoid(w . h + bias), accept when score > theta
 * (strict).  w: [d_model] fp32, host memory (copied).  The hidden state h is the last layer's
 * output after the final RMSNorm.  Until this is called the judge test never fires. */
sj_status sj_load_judge_head(sj_target *t, const float *w_host, float bias, float theta);

/* Runtime switches (for tests and measurements).  Names:
 *   "gemm_impl"  0 = CUDA-core kernels, 1 = tcgen05/TMA kernels (bf16 only; default for bf16)
 *   "attn_impl"  0 = CUDA-core kernel,  1 = tensor-core (mma.sync, fp16 operands) kernel (bf16 models),
 *                2 = tcgen05 kernel (bf16 models, head_dim 128, at most 128 query rows per KV head and sequence, else
 *                it runs as 1); default: 2 at head_dim 128, else 1, for bf16 models; 0 for fp32 models.  The
 *                persistent kernel's attention phase is the tcgen05 one when this is 2, head_dim is 128, a KV
 *                head has at most 64 query rows per sequence, the block has at least 49 rows (its ring stages then
 *                hold a 32 KiB key tile) and the step's caches hold at least "attn_tcgen05_min_tiles" 128-key
 *                tiles per thread block; else the mma.sync one.
 *   "attn_tcgen05_min_tiles"  n >= 0 (default 4; 0 = always): see "attn_impl"
 *   "step_impl"  1 = the whole step as one persistent cooperative kernel (bf16, tcgen05 GEMMs, at most 80
 *                block rows; default when the shape allows), 0 = one kernel per stage
 *   "attn_two_term_layers"  n >= 0 (default 1): in layers [0, n) the tensor-core attention carries queries and
 *                probabilities as a sum of two fp16 terms (twice the MMAs).  Where the residual stream is still
 *                small (the first layer: an embedding row), the attention output is most of what the next
 *                norm sees, and the 2^-11 rounding of one-term operands would dominate the step's error.
 *   "ring_stages" persistent kernel: cap on the shared-memory ring depth (0 = as many as fit, the default)
 *   "trace"      k > 0 = the persistent kernel records a timeline with the nanosecond global timer
 *                (sj_step_trace()): block k - 1 stamps its arrival at and release from every device-wide
 *                barrier and eight events per GEMM phase; every block stamps the first 32 barriers
 *   "graph"      1 = replay the step as a CUDA graph (default unless the stream is NULL, which
 *                cannot be captured), 0 = plain launches
 *   "pdl"        1 = programmatic dependent launch between the step's kernels (default)
 *   "timing"     1 = bracket every kernel launch of a step with CUDA events (needs "graph" 0; turns
 *                programmatic launches off for those steps); setting it (0 or 1) clears old records
 * Errors: INVALID_ARG for an unknown name, UNSUPPORTED for a value the dtype cannot honour. */
sj_status sj_set_option(sj_target *t, const char *name, int value);

/* Device time of the launches recorded under "timing" whose kernel name starts with `name`
 * ("gemm", "gemm_gateup", "attn", "reduce_norm", ...): sum of event-bracketed durations and their
 * count.  Synchronises the stream. */
sj_status sj_kernel_time(sj_target *t, const char *name, double *total_ms, long *launches);

/* Timeline of the last persistent-kernel step run under "trace" (global-timer nanoseconds; unused entries 0).
 * For the traced block: out_ns[2k] is the time it reached device-wide barrier k (k = 1, 2, ... in program
 * order: after the embedding phase, then per layer after QKV, attention, combine, O, gate/up and down, then
 * after the LM head), out_ns[2k+1] the time it was released (k < 1024); out_ns[2048 + 8s + e] is event e of
 * GEMM phase s (s counts QKV, O, gate/up, down per layer, then the LM head): 0 activation loads released,
 * 1 last activation load issued, 2 first stage ready, 3 last MMA issued, 4 last accumulator seen by the
 * epilogue, 5 split-K partial sums gathered, 6 epilogue done, 7 last weight load issued;
 * out_ns[2048 + 4096 + 8s + e] is a second, finer set of epilogue and attention events whose meaning is
 * private to the kernel source.  For every block c < 256 and barrier k < 32: out_ns[10240 + 256k + c] is
 * the block's release time and out_ns[18432 + 256k + c] its arrival time.  Copies at most max_entries
 * (26624 for everything) values into the host array; synchronises the stream. */
sj_status sj_step_trace(sj_target *t, unsigned long long *out_ns, int max_entries, int *n_entries);

/* Wait for the target's stream and return the device status word (SJ_OK, SJ_ERR_TIMEOUT,
 * SJ_ERR_STATE ...), clearing it. */
sj_status sj_sync(sj_target *t);

/* Paged KV cache for up to max_seqs sequences sharing max_pages pages of page_size (16) tokens.
 * A page holds, per layer, K and V rows [Hkv, page_size, head_dim] in the model dtype; keys are
 * stored AFTER the rotary embedding. */
sj_status sj_kv_create(sj_target *t, int max_seqs, long max_pages, int page_size, sj_kv **out);
sj_status sj_kv_destroy(sj_kv *kv);

/* Write n_tokens cache rows of one layer of one sequence starting at token index `start`,
 * reserving pages as needed.  k, v: device, [n_tokens, Hkv, head_dim], model dtype, K already
 * rotated.  Does not change the sequence length.  Errors: OOM (pool exhausted), INVALID_ARG. */
sj_status sj_kv_fill(sj_kv *kv, int seq, int layer, int start, int n_tokens, const void *k, const void *v);
/* Read rows back (same layout); synchronises the stream.  For tests. */
sj_status sj_kv_read(sj_kv *kv, int seq, int layer, int start, int n_tokens, void *k_out, void *v_out);
/* Set the length of sequences (tokens [0,len) are live).  len must not exceed the rows reserved
 * by fills/verifies.  seq_ids, lens: host [B]. */
sj_status sj_kv_set_len(sj_kv *kv, const int *seq_ids, const int *lens, int B);
/* Set the pending token x_t of sequences (fed at row 0 of the next block).  host [B]. */
sj_status sj_kv_set_pending(sj_kv *kv, const int *seq_ids, const int *tokens, int B);
/* Current lengths (host out[B]); synchronises the stream and returns unused pages to the pool. */
sj_status sj_kv_len(sj_kv *kv, const int *seq_ids, int *out_len, int B);

typedef struct {
  int B, gamma;
  const int *seq_ids;        /* host   [B] distinct sequence slots of the sj_kv */
  const int *draft_ids;      /* device [B, gamma]      d_1..d_gamma */
  const float *draft_q_tok;  /* device [B, gamma]      q_j(d_j); required iff mode == SAMPLING */
  const float *draft_q_full; /* device [B, gamma, V]   full draft distributions; required iff SAMPLING */
  const float *uniforms;     /* device [B, gamma+1]    [:, :gamma] = u_1..u_gamma of Eq. 3,
                                                       [:, gamma] drives the emitted token; iff SAMPLING */
  int mode;                  /* SJ_MODE_GREEDY (temperature 0, the paper's setting) or SJ_MODE_SAMPLING */
  float temperature;         /* SAMPLING: p = softmax(logits / temperature), > 0 */
  int use_align, use_judge;  /* which of the two tests may accept (App. D.2 ablation) */
  float theta_override;      /* >= 0: use instead of the loaded theta */
  int commit;                /* 1: kv_len <- kv_len + 1 + accepted_len, pending <- next_token */
  const float *theta_per_seq;/* host [B] or NULL: a judge threshold per sequence (takes precedence; each in [0, 1e30]) */
  int top_k;                 /* GREEDY alignment test: 0 or 1 = the draft must be the target's arg max (strict matching);
                                2 = it must be among the target's two most likely tokens (the top-k baseline of the
                                paper's Sec. 4, k = 2).  Equal logits rank by token id, lowest first */
  int accept_all;            /* 1: accept every drafted position whatever the tests say: the block is a forced
                                continuation (prefill of known tokens, teacher-forced scoring, Eq. 2 alone) */
} sj_verify_args;

typedef struct {
  int *accepted_len;    /* device [B]         n = number of drafts accepted before the first rejection */
  int *next_token;      /* device [B]         greedy: argmax of row n (lowest id on ties); sampling: inverse
                                              CDF (vocab order, uniforms[:,gamma]) of norm(max(0, p_n - q_{n+1}))
                                              when n < gamma, of p_gamma otherwise */
  float *judge_scores;  /* device [B, gamma]  sigmoid scores of d_1..d_gamma (all positions) */
  float *p_draft;       /* device [B, gamma]  p_j(d_j) (at temperature 1 in greedy mode) */
  int *new_kv_len;      /* device [B]         kv_len + 1 + n */
  float *dbg_hidden;    /* device [B, gamma+1, d_model] or NULL: hidden states after the final norm */
  float *dbg_logits;    /* device [B, gamma+1, vocab]   or NULL: raw logits (tests only) */
  float *logp_draft;    /* device [B, gamma] or NULL: log p_j(d_j) (natural log; the teacher-forced log-likelihood
                                              terms of the semantic-preservation score, Eq. 6-7) */
} sj_verify_out;

/* One verification step (see the file comment).  Appends gamma+1 K/V rows per sequence at
 * [kv_len, kv_len+gamma]; with commit the sequence keeps the first 1+n of them.
 * Errors before launch: INVALID_ARG, SHAPE (B*(gamma+1) > max_rows), OOM (page pool), STATE. */
sj_status sj_verify(sj_target *t, sj_kv *kv, const sj_verify_args *args, const sj_verify_out *out);

/* Chunked prefill through the verification step's own kernels: Eq. 2 applied to tokens that are known
 * rather than drafted.  Appends the n_tokens tokens `tokens` (host) to sequence `seq` in blocks of up to
 * min(32, 96 / (Hq/Hkv), max_rows) tokens: each block runs as a verification step whose first row is the
 * block's first token and whose "drafts" are the following ones, every position accepted and committed
 * (accept_all), so the cache receives exactly the K/V rows a verification step would read.  On return (the
 * work is queued on the target's stream) the sequence is n_tokens longer and its pending token is the target's
 * greedy token after the last appended one; with next_token != NULL (host) that token is also copied out,
 * which waits for the stream.  The sequence's previous pending token is dropped: the first appended token
 * takes its place.  Errors: INVALID_ARG, SHAPE, OOM (page pool), and whatever sj_verify() reports. */
sj_status sj_prefill(sj_target *t, sj_kv *kv, int seq, const int *tokens, int n_tokens, int *next_token);

/* Semantic-preservation score of a token replacement (Sec. 3.3, Eq. 6 in the autoregressive form of Eq. 7):
 *   s = [log P(z_i | y_<i) - log P(y_i | y_<i)]
 *       + sum_{k=1..N} [log P(y_{i+k} | y_<i, z_i, y_{i+1..i+k-1}) - log P(y_{i+k} | y_<i, y_i, y_{i+1..i+k-1})]
 * the quantity whose threshold labels the verifier's training tokens.  Sequence `seq` must hold y_{<i-1} in the
 * cache and y_{i-1} as its pending token; `future` (host) are the N = n_future <= 30 tokens y_{i+1..i+N}.  Two
 * uncommitted verification steps over [y_{i-1}; z_i or y_i, future...] give the teacher-forced log-probabilities
 * (sj_verify_out.logp_draft); the cache, the length and the pending token are left as they were.
 * score (host, two floats): s and its prefix term log P(z_i | y_<i) - log P(y_i | y_<i).  Waits for the stream.
 * Errors: INVALID_ARG, SHAPE, and whatever sj_verify() reports. */
sj_status sj_semantic_score(sj_target *t, sj_kv *kv, int seq, int y_i, int z_i, const int *future, int n_future,
                            float *score);

/* Truncate sequences to new_len <= current length (host arrays [B]) and return the whole pages
 * past new_len to the pool (the KV-length rollback that follows the first-rejection scan, Sec. 3.1).
 * Asynchronous; if new_len exceeds the true length the device leaves the sequence unchanged and
 * sj_sync() returns SJ_ERR_STATE.  new_len above what the host knows could be live fails at once
 * with STATE. */
sj_status sj_rollback_kv(sj_kv *kv, const int *seq_ids, const int *new_len, int B);

/* Skinny GEMM used by every projection of the step, exposed for kernel-level tests and
 * measurement:  y[R, N] (fp32) = a[R, K] . w[N, K]^T,  a and w in `dtype`, device pointers.
 * impl as in "gemm_impl".  Synchronous with respect to `cuda_stream` ordering only. */
sj_status sj_gemm_skinny(int dtype, int impl, int R, int N, int K, const void *a, const void *w, float *y,
                         void *cuda_stream);

/* The same product as sj_gemm_skinny(SJ_DTYPE_BF16, impl 1, ...), for callers that must not allocate.
 * (The paper has no counterpart to this call; it exists for the library's users.)
 *
 * Who needs it: code that runs where device allocation is forbidden or unsafe -- inside a serving
 * engine that has handed all of the GPU's memory to its own pool, while another thread is capturing a
 * stream (cudaMalloc and cudaFree are illegal during a capture and break it), or on a latency path
 * where the implicit device synchronisation of cudaFree cannot be afforded.  sj_gemm_skinny() takes
 * its split-K partial-sum buffer from cudaMalloc on every call; this variant keeps that buffer in a
 * fixed array of SJ_NOALLOC_SCRATCH_BYTES that is part of the library image.  Every GPU on which the
 * library's kernels are loaded holds those bytes until the process exits, used or not.
 *
 *   y[R, N] (fp32) = a[R, K] . w[N, K]^T,  a and w bf16, row-major, 16-byte aligned device pointers,
 *   K a multiple of 64.  The caller owns a, w and y.  Work is queued on `cuda_stream` and the call
 *   returns after that stream has drained (it reads back the device status word).
 *
 * Size limit: 256 + round_up(8 * T, 256) + 4 * slots * R * N bytes must fit in the array, with
 * T = ceil(N/128) tiles and slots = the largest number of thread blocks that share one tile's K range:
 * the T * (K/64) work units are dealt evenly to G = min(#SMs, T * K/64) blocks, so
 * slots <= ceil((K/64) / floor(T * (K/64) / G)) + 1.  Larger problems are refused with SJ_ERR_SHAPE and
 * a message naming the bytes needed; nothing is launched.
 *
 * The first call on each device resolves the array's device address (cudaGetSymbolAddress, with that
 * device current) and opts the kernel into its shared-memory size; make that first call outside any
 * stream capture.  No call allocates or frees device memory or calls a routine that does.
 *
 * All calls on one device share the array, and it keeps whatever the previous call left: each call
 * zeroes the status word and rewrites the slot table and every partial sum before reading them.
 * Two calls whose kernels overlap on the GPU (different streams, or different host threads) race on
 * that memory and give wrong results: serialise them.
 * Errors: INVALID_ARG (null), SHAPE (sizes, scratch limit), UNSUPPORTED (not sm_100), CUDA, TIMEOUT. */
enum { SJ_NOALLOC_SCRATCH_BYTES = 8 * 1024 * 1024 };
sj_status sj_gemm_skinny_noalloc(int R, int N, int K, const void *a, const void *w, float *y, void *cuda_stream);

/* Fault drill without a fault (the paper has no counterpart).  Every device-side wait of the library is
 * bounded: when one runs out, the kernel records the fact, returns normally, and the next sj_sync() reports
 * SJ_ERR_TIMEOUT; the context stays usable.  This call queues, on the target's stream, a one-block kernel
 * that runs that same wait code on a barrier (kind 0: the stand-alone GEMM kernels' wait; kind 1: the ring /
 * accumulator wait of the attention and whole-step kernels) or a device-memory word (kind 2: the whole-step
 * kernel's device-wide barrier poll) that nothing will ever signal, with a limit of max_polls (1 .. 2^20)
 * polls.  Use it to exercise an application's handling of SJ_ERR_TIMEOUT.  Nothing traps, faults or hangs.
 * Errors: INVALID_ARG, UNSUPPORTED (the target was created without the whole-step kernel's workspace). */
sj_status sj_debug_expire_wait(sj_target *t, int kind, unsigned max_polls);

/* How many device-memory allocation and release calls (cudaMalloc / cudaFree) the library has made in this
 * process so far.  Diagnostic (the paper has no counterpart): lets a caller check that a call it relies on
 * to be allocation-free, such as sj_gemm_skinny_noalloc() or a steady-state sj_verify(), really made none. */
long sj_device_memory_calls(void);

const char *sj_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SJ_H_ */
