// Shared device-side definitions for the verification-step kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sj {

typedef __nv_bfloat16 bf16;

constexpr int kMaxBatch = 256;
constexpr int kMaxGamma = 31;
constexpr int kMaxRows = 512;
constexpr int kTileN = 128;  // output features per GEMM tile (the MMA's M after swapping operands)

// device status word values (first error wins)
enum DevStatus { DEV_OK = 0, DEV_TIMEOUT = 7, DEV_STATE = 3 };

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(bf16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float x) { return __float2bfloat16_rn(x); }

// Per-call arguments, resident in device memory and rewritten by one small copy per call so
// that a captured graph never bakes in a caller's pointer.
struct StepArgs {
  const int* draft_ids;
  const float* q_tok;
  const float* q_full;
  const float* uniforms;
  int* accepted_len;
  int* next_token;
  float* judge_scores;
  float* p_draft;
  int* new_kv_len;
  float* dbg_hidden;
  float* dbg_logits;
  float* logp_draft;      // optional: natural log of p_j(d_j)
  int B, gamma, mode, use_align, use_judge, commit;
  int top_k;              // greedy alignment test: the draft must be among the target's top_k tokens (1 or 2)
  int accept_all;         // every drafted position is accepted whatever the tests say (prefill, teacher forcing)
  float inv_temperature, judge_bias;
  int has_judge;
  int seq_ids[kMaxBatch];
  float theta[kMaxBatch]; // judge threshold per sequence of the batch
};

// Paged KV cache view.  Element (layer, page, kv in {0,1}, head, slot, dim):
//   pool[((((layer * n_pages + page) * 2 + kv) * Hkv + head) * page_size + slot) * hd + dim]
struct KvView {
  void* pool;
  const int* block_table;  // [max_seqs, max_pages_per_seq]
  int* kv_len;             // [max_seqs]
  int* pending;            // [max_seqs]
  long n_pages;
  int max_pages_per_seq;
  int page_size;           // 16
  int n_kv_heads, head_dim;
};

template <typename T>
__device__ __forceinline__ T* kv_row(const KvView& kv, int layer, int page, int which, int head, int slot) {
  size_t idx = ((((size_t)layer * kv.n_pages + page) * 2 + which) * kv.n_kv_heads + head);
  idx = (idx * kv.page_size + slot) * kv.head_dim;
  return reinterpret_cast<T*>(kv.pool) + idx;
}

// How a GEMM's output tile is spread over thread blocks (split along K).  Work is counted in
// units of (128-feature tile, 64-wide K block); block c owns units [c*U/G, (c+1)*U/G).  A tile's
// partial sums live in consecutive "slots" of the partial buffer, one per contributing block in
// block order, so that the consumer adds them in a fixed order (no atomics, bit-reproducible).
struct SplitPlan {
  const int2* tile_slots;  // per tile: (first contributing block, number of slots); null: one slot
  int n_tiles;
};

// Partial buffer layout: P[slot][row][N] fp32.
__device__ __forceinline__ float reduce_partials(const float* __restrict__ P, const SplitPlan& sp, size_t slot_stride,
                                                 int N, int r, int n) {
  const float* p = P + (size_t)r * N + n;
  if (sp.tile_slots == nullptr) return *p;
  int cnt = sp.tile_slots[n / kTileN].y;
  float s = 0.f;
  for (int i = 0; i < cnt; ++i) s += p[(size_t)i * slot_stride];
  return s;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum with a fixed reduction tree (deterministic).  `red` holds >= 32 floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  float t = (threadIdx.x < nw) ? red[threadIdx.x] : 0.f;
  if (w == 0) {
    t = warp_sum(t);
    if (lane == 0) red[0] = t;
  }
  __syncthreads();
  return red[0];
}

// Programmatic dependent launch: every kernel of the step calls pdl_wait() before it reads or
// writes anything another kernel of the step produces, and pdl_launch() once its own dependents
// may be scheduled.  Both are no-ops when the launch carries no programmatic dependency.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Softmax statistics of a set of logits: running maximum m, sum of exp(z - m), arg max.
struct RowStat {
  float m, s;
  int arg;
  int pad;   // top-k test: how many of the set's logits rank before the drafted token's (larger, or equal with a lower id)
};
__device__ __forceinline__ RowStat stat_merge(const RowStat& a, const RowStat& b) {
  // a precedes b in vocabulary order: on equal maxima the lower index (a) is kept
  RowStat r;
  bool take_b = b.m > a.m;
  r.m = take_b ? b.m : a.m;
  r.arg = take_b ? b.arg : a.arg;
  float sa = (a.m == -INFINITY) ? 0.f : a.s * expf(a.m - r.m);
  float sb = (b.m == -INFINITY) ? 0.f : b.s * expf(b.m - r.m);
  r.s = sa + sb;
  r.pad = a.pad + b.pad;
  return r;
}

}  // namespace sj
