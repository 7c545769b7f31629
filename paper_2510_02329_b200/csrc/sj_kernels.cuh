// Elementwise, CUDA-core GEMM / attention, LM-head statistics and acceptance kernels of the
// verification step.  Templated on the storage type T (float or bf16); accumulation is fp32.
#pragma once

#include "sj_common.cuh"

namespace sj {

// Device workspace of one target (all sized for max_rows).
struct Work {
  float* X;          // [R, d]        fp32 residual stream
  // GEMM inputs.  fp32 models: one plane [R, K] of floats.  bf16 models: TWO bf16 planes
  // [2][Rp][K] (Rp = R rounded up to 16): plane 0 holds bf16(x), plane 1 holds bf16(x - plane 0), so
  // that the tensor cores see x to ~2^-17 instead of 2^-9; the product with both planes is summed
  // in the fp32 accumulator's epilogue.
  void* A;           // normalised activations (input of QKV / gate-up / LM head), K = d
  float* Q;          // [R, Hq*hd]    fp32 rotated queries
  __half* Qb;        // [B, Hkv, group*(gamma+1), hd] fp16 rotated queries times log2(e)/sqrt(hd), query row
                     // g*(gamma+1)+j of a KV head's group (tensor-core attention), or null
  __half* Qlo;       // same layout: what the fp16 rounding of Qb dropped (q - Qb, rounded to fp16), for the layers in
                     // which the attention runs with two-term operands
  __half* KVn;       // [B, Hkv, 2 (K|V), gamma+1, hd] fp16 copy of this step's own key / value rows (the rows the
                     // pages receive in bf16): the tensor-core attention reads the block's own rows from here
  void* ATT;         // attention output (input of the O projection), K = Hq*hd
  void* H;           // silu(gate)*up (input of the down projection), K = F
  float* P;          // partial sums of the current GEMM: [slot][R][N]
  float* Hf;         // [R, d]        fp32 hidden state after the final norm
  float2* rope;      // [R, hd/2]     (cos, sin) of this step's positions
  int* row_pos;      // [R]           absolute position of each row
  int* chunk_start;  // [B+1]         prefix sum of attention chunks per sequence
  float* att_m;      // [chunks, Hq, gamma+1]         running max of each partial
  float* att_l;      // same                           sum of exp
  float* att_o;      // [chunks, Hq, gamma+1, hd]      unnormalised partial outputs
  float* tc_m;       // tensor-core attention partials: [slots][4][nq] running max (log2 domain)
  float* tc_l;       // same                            sum of exp2
  float* tc_o;       // [slots][4][nq][hd]              unnormalised outputs
  RowStat* stats;    // [vocab tiles, R]
  float* tgt_logit;  // [R]   logit of the drafted token d_{j+1} in row j
  float* tgt_pre;    // [R]   the same logit (raw), computed BEFORE the LM head when the top-k test needs it to count ranks
  RowStat* rowstat;  // [R]   merged statistics
  float* logits;     // fp32 logit scratch, or null: [R, V] for the CUDA-core LM head; [B, V] in sampling mode with
                     // the tensor-core LM head (only the one row per sequence that the emitted token is drawn from)
  void* Asel;        // GEMM input planes of those B rows (final-norm hidden states), K = d
  const double* inv_freq;  // [hd/2] rope_theta^(-2i/hd)
  const float* judge_w;    // [d]
  int* status;
};

struct Dims {
  int n_layers, d, Hq, Hkv, hd, F, V;
  float eps;
};

__host__ __device__ __forceinline__ int pad16(int r) { return (r + 15) & ~15; }

// Store one GEMM-input element (row r of R, column i of K).
template <typename T> __device__ __forceinline__ void store_act(void* base, int R, int K, int r, int i, float y);
template <> __device__ __forceinline__ void store_act<float>(void* base, int R, int K, int r, int i, float y) {
  reinterpret_cast<float*>(base)[(size_t)r * K + i] = y;
}
template <> __device__ __forceinline__ void store_act<bf16>(void* base, int R, int K, int r, int i, float y) {
  bf16 hi = __float2bfloat16_rn(y);
  bf16 lo = __float2bfloat16_rn(y - __bfloat162float(hi));
  bf16* b = reinterpret_cast<bf16*>(base);
  b[(size_t)r * K + i] = hi;
  b[((size_t)pad16(R) + r) * K + i] = lo;
}

// ---------------------------------------------------------------------------------------------
// step set-up: row positions and the attention chunk list (needs the true cache lengths)
// ---------------------------------------------------------------------------------------------
__global__ void k_plan(const StepArgs* __restrict__ args, KvView kv, Work w, int chunk_len) {
  pdl_wait();
  pdl_launch();
  __shared__ int nch[kMaxBatch];
  const int B = args->B, rows = args->gamma + 1;
  for (int b = threadIdx.x; b < B; b += blockDim.x) {
    int L = kv.kv_len[args->seq_ids[b]];
    nch[b] = (L + rows + chunk_len - 1) / chunk_len;
    for (int j = 0; j < rows; ++j) w.row_pos[b * rows + j] = L + j;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int b = 0; b < B; ++b) {
      w.chunk_start[b] = acc;
      acc += nch[b];
    }
    w.chunk_start[B] = acc;
  }
}

// RMSNorm of a row held in shared memory; writes T activations and optional fp32 copies.
template <typename T>
__device__ __forceinline__ void norm_row_from_smem(const float* xs, int d, const T* __restrict__ gain, float eps,
                                                   void* act, int R, int r, float* hf_row, float* dbg_row, float* red) {
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) ss += xs[i] * xs[i];
  ss = block_sum(ss, red);
  float inv = 1.0f / sqrtf(ss / (float)d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float y = xs[i] * inv * to_f(gain[i]);
    store_act<T>(act, R, d, r, i, y);
    if (hf_row) hf_row[i] = y;
    if (dbg_row) dbg_row[i] = y;
  }
}

// a1 + first a2: embedding gather, RMSNorm, and this step's rotary table.
template <typename T>
__global__ void k_embed_norm(const StepArgs* __restrict__ args, KvView kv, Work w, Dims dm, const T* __restrict__ embed,
                             const T* __restrict__ gain) {
  extern __shared__ float xs[];
  __shared__ float red[32];
  pdl_wait();
  pdl_launch();
  const int r = blockIdx.x, rows = args->gamma + 1;
  const int b = r / rows, j = r % rows;
  const int seq = args->seq_ids[b];
  int tok = (j == 0) ? kv.pending[seq] : args->draft_ids[b * args->gamma + j - 1];
  tok = min(max(tok, 0), dm.V - 1);
  const T* e = embed + (size_t)tok * dm.d;
  for (int i = threadIdx.x; i < dm.d; i += blockDim.x) {
    float x = to_f(e[i]);
    xs[i] = x;
    w.X[(size_t)r * dm.d + i] = x;
  }
  const int pos = kv.kv_len[seq] + j;
  for (int i = threadIdx.x; i < dm.hd / 2; i += blockDim.x) {
    double s, c;
    sincos((double)pos * w.inv_freq[i], &s, &c);
    w.rope[(size_t)r * (dm.hd / 2) + i] = make_float2((float)c, (float)s);
  }
  __syncthreads();
  norm_row_from_smem<T>(xs, dm.d, gain, dm.eps, w.A, gridDim.x, r, nullptr, nullptr, red);
}

// a6/a8 tail + a2/a9: X += sum of partials; A = RMSNorm(X) * gain.  final: also fp32 hidden.
template <typename T>
__global__ void k_reduce_norm(const StepArgs* __restrict__ args, Work w, Dims dm, SplitPlan sp, size_t slot_stride,
                              const T* __restrict__ gain, int final_norm) {
  extern __shared__ float xs[];
  __shared__ float red[32];
  pdl_wait();
  pdl_launch();
  const int r = blockIdx.x;
  for (int i = threadIdx.x; i < dm.d; i += blockDim.x) {
    float x = w.X[(size_t)r * dm.d + i] + reduce_partials(w.P, sp, slot_stride, dm.d, r, i);
    xs[i] = x;
    w.X[(size_t)r * dm.d + i] = x;
  }
  __syncthreads();
  float* hf = final_norm ? w.Hf + (size_t)r * dm.d : nullptr;
  float* dbg = (final_norm && args->dbg_hidden) ? args->dbg_hidden + (size_t)r * dm.d : nullptr;
  norm_row_from_smem<T>(xs, dm.d, gain, dm.eps, w.A, gridDim.x, r, hf, dbg, red);
}

// a3 tail + a4: reduce QKV partials, add bias, rotate q and k, store q, append k and v rows.
template <typename T>
__global__ void k_qkv_rope(const StepArgs* __restrict__ args, KvView kv, Work w, Dims dm, SplitPlan sp,
                           size_t slot_stride, int layer, const T* __restrict__ bq, const T* __restrict__ bk,
                           const T* __restrict__ bv) {
  pdl_wait();
  pdl_launch();
  const int r = blockIdx.x, rows = args->gamma + 1;
  const int b = r / rows;
  const int seq = args->seq_ids[b];
  const int pos = w.row_pos[r];
  const int half = dm.hd / 2;
  const int qd = dm.Hq * dm.hd, kd = dm.Hkv * dm.hd, N = qd + 2 * kd;
  const int page = kv.block_table[(size_t)seq * kv.max_pages_per_seq + pos / kv.page_size];
  const int slot = pos % kv.page_size;
  const float2* rt = w.rope + (size_t)r * half;
  // rotated heads: q heads then k heads
  for (int p = threadIdx.x; p < (dm.Hq + dm.Hkv) * half; p += blockDim.x) {
    int head = p / half, i = p % half;
    int n1 = head * dm.hd + i, n2 = n1 + half;
    float x1 = reduce_partials(w.P, sp, slot_stride, N, r, n1);
    float x2 = reduce_partials(w.P, sp, slot_stride, N, r, n2);
    if (head < dm.Hq) {
      if (bq) { x1 += to_f(bq[n1]); x2 += to_f(bq[n2]); }
    } else if (bk) {
      x1 += to_f(bk[n1 - qd]); x2 += to_f(bk[n2 - qd]);
    }
    float2 cs = rt[i];
    float y1 = x1 * cs.x - x2 * cs.y;
    float y2 = x2 * cs.x + x1 * cs.y;
    if (head < dm.Hq) {
      float* q = w.Q + (size_t)r * qd;
      q[n1] = y1;
      q[n2] = y2;
      if (w.Qb) {
        const int group = dm.Hq / dm.Hkv, j = r % rows;
        const float qs = 1.4426950408889634f / sqrtf((float)dm.hd);
        __half* qb = w.Qb + ((((size_t)b * dm.Hkv + head / group) * group + head % group) * rows + j) * dm.hd;
        const __half h1 = __float2half_rn(y1 * qs), h2 = __float2half_rn(y2 * qs);
        qb[i] = h1;
        qb[i + half] = h2;
        __half* ql = w.Qlo + (qb - w.Qb);
        ql[i] = __float2half_rn(y1 * qs - __half2float(h1));
        ql[i + half] = __float2half_rn(y2 * qs - __half2float(h2));
      }
    } else {
      T* krow = kv_row<T>(kv, layer, page, 0, head - dm.Hq, slot);
      krow[i] = from_f<T>(y1);
      krow[i + half] = from_f<T>(y2);
      if (w.KVn) {
        __half* kn = w.KVn + ((((size_t)b * dm.Hkv + head - dm.Hq) * 2) * rows + r % rows) * dm.hd;
        kn[i] = __float2half_rn(y1);
        kn[i + half] = __float2half_rn(y2);
      }
    }
  }
  for (int p = threadIdx.x; p < kd; p += blockDim.x) {
    float x = reduce_partials(w.P, sp, slot_stride, N, r, qd + kd + p);
    if (bv) x += to_f(bv[p]);
    T* vrow = kv_row<T>(kv, layer, page, 1, p / dm.hd, slot);
    vrow[p % dm.hd] = from_f<T>(x);
    if (w.KVn) w.KVn[((((size_t)b * dm.Hkv + p / dm.hd) * 2 + 1) * rows + r % rows) * dm.hd + p % dm.hd] = __float2half_rn(x);
  }
}

// a7 tail: H = silu(gate) * up from the partials of the fused [gate; up] projection.
template <typename T>
__global__ void k_swiglu(Work w, Dims dm, SplitPlan sp, size_t slot_stride) {
  pdl_wait();
  pdl_launch();
  const int r = blockIdx.y;
  const int f = blockIdx.x * blockDim.x + threadIdx.x;
  if (f >= dm.F) return;
  float g = reduce_partials(w.P, sp, slot_stride, 2 * dm.F, r, f);
  float u = reduce_partials(w.P, sp, slot_stride, 2 * dm.F, r, dm.F + f);
  float y = g / (1.0f + expf(-g)) * u;
  store_act<T>(w.H, gridDim.y, dm.F, r, f, y);
}

// ---------------------------------------------------------------------------------------------
// CUDA-core skinny GEMM: one warp per output feature, RT rows at a time.  Used for fp32 models
// and as a cross-check of the tensor-core kernel.
// ---------------------------------------------------------------------------------------------
struct GemmSegs {
  const void* w[3];  // up to three weight matrices stacked along the output dimension
  int rows[3];
  int nseg;
};

template <typename T> struct Vec;
template <> struct Vec<float> { typedef float4 type; static constexpr int n = 4; };
template <> struct Vec<bf16> { typedef uint4 type; static constexpr int n = 8; };

__device__ __forceinline__ void unpack(const float4& v, float* f) { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
__device__ __forceinline__ void unpack(const uint4& v, float* f) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __bfloat1622float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

// `planes` = 2: the input is a hi/lo pair of bf16 planes (see Work); the two are added before use.
template <typename T, int RT>
__global__ void k_gemm_simt(const T* __restrict__ A, GemmSegs segs, float* __restrict__ Y, int R, int N, int K,
                            int planes) {
  pdl_wait();
  pdl_launch();
  constexpr int VN = Vec<T>::n;
  typedef typename Vec<T>::type V;
  const int lane = threadIdx.x & 31;
  const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (n >= N) return;
  int nn = n, s = 0;
  while (s < segs.nseg - 1 && nn >= segs.rows[s]) { nn -= segs.rows[s]; ++s; }
  const T* wrow = reinterpret_cast<const T*>(segs.w[s]) + (size_t)nn * K;
  for (int r0 = 0; r0 < R; r0 += RT) {
    float acc[RT];
#pragma unroll
    for (int i = 0; i < RT; ++i) acc[i] = 0.f;
    for (int k = lane * VN; k < K; k += 32 * VN) {
      float wf[VN];
      unpack(*reinterpret_cast<const V*>(wrow + k), wf);
#pragma unroll
      for (int i = 0; i < RT; ++i) {
        if (r0 + i < R) {
          float af[VN];
          unpack(*reinterpret_cast<const V*>(A + (size_t)(r0 + i) * K + k), af);
          if (planes == 2) {
            float lo[VN];
            unpack(*reinterpret_cast<const V*>(A + ((size_t)pad16(R) + r0 + i) * K + k), lo);
#pragma unroll
            for (int e = 0; e < VN; ++e) af[e] += lo[e];
          }
#pragma unroll
          for (int e = 0; e < VN; ++e) acc[i] = fmaf(af[e], wf[e], acc[i]);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < RT; ++i) {
      float v = warp_sum(acc[i]);
      if (lane == 0 && r0 + i < R) Y[(size_t)(r0 + i) * N + n] = v;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// a5: causal grouped-query attention over the paged cache, split along the keys.
// Work item = (chunk of chunk_len keys of one sequence, KV head); all query heads of the group and
// all gamma+1 rows share the item's K/V.  Each item writes unnormalised partials (m, l, o).
// ---------------------------------------------------------------------------------------------
constexpr int kAttKT = 32;      // keys per inner tile
constexpr int kAttMaxQ = 96;    // query vectors per item: (Hq/Hkv) * (gamma+1)
constexpr int kAttThreads = 256;

__device__ __forceinline__ int find_seq(const int* chunk_start, int B, int chunk) {
  int lo = 0, hi = B - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (chunk_start[mid] <= chunk) lo = mid; else hi = mid - 1;
  }
  return lo;
}

template <typename T>
__global__ void k_attn_simt(const StepArgs* __restrict__ args, KvView kv, Work w, Dims dm, int layer, int chunk_len) {
  extern __shared__ float sm[];
  pdl_wait();
  pdl_launch();
  const int B = args->B, rows = args->gamma + 1;
  const int group = dm.Hq / dm.Hkv, nq = group * rows, hd = dm.hd;
  float* qs = sm;                         // [nq][hd]
  float* ks = qs + nq * hd;               // [KT][hd+1]
  float* vs = ks + kAttKT * (hd + 1);     // [KT][hd]
  float* ss = vs + kAttKT * hd;           // [nq][KT]
  float* m_run = ss + nq * kAttKT;        // [nq]
  float* l_run = m_run + nq;              // [nq]
  float* alpha = l_run + nq;              // [nq]
  const float scale = 1.0f / sqrtf((float)hd);
  const int total = w.chunk_start[B] * dm.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int item = blockIdx.x; item < total; item += gridDim.x) {
    const int chunk = item / dm.Hkv, kvh = item % dm.Hkv;
    const int b = find_seq(w.chunk_start, B, chunk);
    const int seq = args->seq_ids[b];
    const int L = w.row_pos[b * rows];  // cached tokens before the block
    const int k_begin = (chunk - w.chunk_start[b]) * chunk_len;
    const int k_end = min(k_begin + chunk_len, L + rows);
    __syncthreads();
    // queries of this KV head's group: q index = g * rows + j
    for (int i = tid; i < nq * hd; i += kAttThreads) {
      int q = i / hd, dd = i % hd, g = q / rows, j = q % rows;
      const float* qrow = w.Q + (size_t)(b * rows + j) * (dm.Hq * hd) + (kvh * group + g) * hd;
      qs[i] = qrow[dd];
    }
    for (int q = tid; q < nq; q += kAttThreads) { m_run[q] = -INFINITY; l_run[q] = 0.f; }
    float acc[48];
#pragma unroll
    for (int i = 0; i < 48; ++i) acc[i] = 0.f;
    for (int k0 = k_begin; k0 < k_end; k0 += kAttKT) {
      __syncthreads();
      for (int i = tid; i < kAttKT * hd; i += kAttThreads) {
        int kk = i / hd, dd = i % hd, key = k0 + kk;
        float kvv = 0.f, vvv = 0.f;
        if (key < k_end) {
          int page = kv.block_table[(size_t)seq * kv.max_pages_per_seq + key / kv.page_size];
          int slot = key % kv.page_size;
          kvv = to_f(kv_row<T>(kv, layer, page, 0, kvh, slot)[dd]);
          vvv = to_f(kv_row<T>(kv, layer, page, 1, kvh, slot)[dd]);
        }
        ks[kk * (hd + 1) + dd] = kvv;
        vs[kk * hd + dd] = vvv;
      }
      __syncthreads();
      // scores: one (q, key) pair per thread-iteration; a warp covers the 32 keys of one q
      for (int p = tid; p < nq * kAttKT; p += kAttThreads) {
        int q = p / kAttKT, kk = p % kAttKT, key = k0 + kk, j = q % rows;
        float s = -INFINITY;
        if (key < k_end && key <= L + j) {
          float a = 0.f;
          const float* qv = qs + q * hd;
          const float* kvp = ks + kk * (hd + 1);
          for (int dd = 0; dd < hd; ++dd) a = fmaf(qv[dd], kvp[dd], a);
          s = a * scale;
        }
        ss[p] = s;
      }
      __syncthreads();
      // online softmax, one warp per query vector
      for (int q = warp; q < nq; q += kAttThreads / 32) {
        float s = ss[q * kAttKT + lane];
        float mx = warp_max(s);
        float m_old = m_run[q];
        float m_new = fmaxf(m_old, mx);
        float p = (s == -INFINITY) ? 0.f : expf(s - m_new);
        float sum = warp_sum(p);
        ss[q * kAttKT + lane] = p;
        if (lane == 0) {
          float a = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
          alpha[q] = (m_new == -INFINITY) ? 1.f : a;
          l_run[q] = l_run[q] * ((m_new == -INFINITY) ? 1.f : a) + sum;
          m_run[q] = m_new;
        }
      }
      __syncthreads();
      // o[q][dd] = o * alpha + sum_k p[q][k] v[k][dd]
#pragma unroll
      for (int i = 0; i < 48; ++i) {
        int e = tid + i * kAttThreads;
        if (e < nq * hd) {
          int q = e / hd, dd = e % hd;
          float a = acc[i] * alpha[q];
          const float* pv = ss + q * kAttKT;
#pragma unroll 8
          for (int kk = 0; kk < kAttKT; ++kk) a = fmaf(pv[kk], vs[kk * hd + dd], a);
          acc[i] = a;
        }
      }
    }
    __syncthreads();
    // partials: index ((chunk * Hq + head) * rows + j)
#pragma unroll
    for (int i = 0; i < 48; ++i) {
      int e = tid + i * kAttThreads;
      if (e < nq * hd) {
        int q = e / hd, dd = e % hd, g = q / rows, j = q % rows;
        size_t pi = ((size_t)chunk * dm.Hq + kvh * group + g) * rows + j;
        w.att_o[pi * hd + dd] = acc[i];
      }
    }
    for (int q = tid; q < nq; q += kAttThreads) {
      int g = q / rows, j = q % rows;
      size_t pi = ((size_t)chunk * dm.Hq + kvh * group + g) * rows + j;
      w.att_m[pi] = m_run[q];
      w.att_l[pi] = l_run[q];
    }
  }
}

// Merge the partials of one (row, head) over its sequence's chunks, in chunk order.
template <typename T>
__global__ void k_attn_combine(const StepArgs* __restrict__ args, Work w, Dims dm) {
  pdl_wait();
  pdl_launch();
  const int rows = args->gamma + 1;
  const int r = blockIdx.x / dm.Hq, h = blockIdx.x % dm.Hq;
  const int b = r / rows, j = r % rows;
  const int c0 = w.chunk_start[b], c1 = w.chunk_start[b + 1];
  float M = -INFINITY;
  for (int c = c0; c < c1; ++c) M = fmaxf(M, w.att_m[((size_t)c * dm.Hq + h) * rows + j]);
  float Lsum = 0.f;
  for (int c = c0; c < c1; ++c) {
    size_t pi = ((size_t)c * dm.Hq + h) * rows + j;
    float m = w.att_m[pi];
    if (m != -INFINITY) Lsum += w.att_l[pi] * expf(m - M);
  }
  for (int dd = threadIdx.x; dd < dm.hd; dd += blockDim.x) {
    float o = 0.f;
    for (int c = c0; c < c1; ++c) {
      size_t pi = ((size_t)c * dm.Hq + h) * rows + j;
      float m = w.att_m[pi];
      if (m != -INFINITY) o += w.att_o[pi * dm.hd + dd] * expf(m - M);
    }
    store_act<T>(w.ATT, gridDim.x / dm.Hq, dm.Hq * dm.hd, r, h * dm.hd + dd, o / Lsum);
  }
}

// Dot product of GEMM-input row r (both bf16 planes) with one weight row, over the whole warp.
__device__ __forceinline__ float planes_dot(const bf16* __restrict__ A, int R, int K, int r, const bf16* __restrict__ wrow,
                                            int lane) {
  const bf16* hi = A + (size_t)r * K;
  const bf16* lo = A + ((size_t)pad16(R) + r) * K;
  float acc = 0.f;
  for (int k = lane; k < K; k += 32) acc = fmaf(__bfloat162float(hi[k]) + __bfloat162float(lo[k]), __bfloat162float(wrow[k]), acc);
  return warp_sum(acc);
}

// Top-k alignment test with the tensor-core LM head, which stores no logits: the logit of row j's drafted token
// d_{j+1} is computed ahead of the LM head (one dot product per row), so that the head's epilogue can count, tile
// by tile, how many logits rank before it.  One warp per row; idle unless the step asks for top_k >= 2.
__global__ void k_target_logits(const StepArgs* __restrict__ args, Work w, Dims dm, const bf16* __restrict__ lm_head, int R) {
  pdl_wait();
  pdl_launch();
  if (args->top_k < 2) return;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= R) return;
  const int rows = args->gamma + 1, b = r / rows, j = r % rows;
  if (j >= args->gamma) return;
  const int tok = min(max(args->draft_ids[b * args->gamma + j], 0), dm.V - 1);
  const float z = planes_dot(reinterpret_cast<const bf16*>(w.A), R, dm.d, r, lm_head + (size_t)tok * dm.d, lane);
  if (lane == 0) w.tgt_pre[r] = z;
}

// ---------------------------------------------------------------------------------------------
// a10 (CUDA-core path): per-(128-token vocabulary tile, row) softmax statistics from stored logits
// ---------------------------------------------------------------------------------------------
__global__ void k_lm_stats_from_logits(const StepArgs* __restrict__ args, Work w, Dims dm, int R) {
  pdl_wait();
  pdl_launch();
  const int tile = blockIdx.x, lane = threadIdx.x & 31;
  const int r = blockIdx.y * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= R) return;
  const int rows = args->gamma + 1, b = r / rows, j = r % rows;
  const float invT = args->inv_temperature;
  const float* lg = w.logits + (size_t)r * dm.V;
  const int tgt = (j < args->gamma) ? args->draft_ids[b * args->gamma + j] : -1;
  float z[4];
  float m = -INFINITY;
  int arg = 0x7fffffff;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int v = tile * kTileN + i * 32 + lane;
    float raw = (v < dm.V) ? lg[v] : -INFINITY;
    if (v < dm.V && args->dbg_logits) args->dbg_logits[(size_t)r * dm.V + v] = raw;
    z[i] = raw * invT;
    if (v == tgt) w.tgt_logit[r] = z[i];
    if (z[i] > m) { m = z[i]; arg = v; }   // increasing v: strict > keeps the lowest index
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float om = __shfl_xor_sync(0xffffffffu, m, o);
    int oa = __shfl_xor_sync(0xffffffffu, arg, o);
    if (om > m || (om == m && oa < arg)) { m = om; arg = oa; }
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) s += (z[i] == -INFINITY) ? 0.f : expf(z[i] - m);
  s = warp_sum(s);
  int before = 0;   // top-k test: this tile's logits that rank before the drafted token's (the logits are stored here)
  if (args->top_k >= 2 && tgt >= 0) {
    const float zd = lg[min(tgt, dm.V - 1)];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int v = tile * kTileN + i * 32 + lane;
      const float raw = (v < dm.V) ? lg[v] : -INFINITY;
      const bool bf = v < dm.V && v != tgt && (raw > zd || (raw == zd && v < tgt));
      before += __popc(__ballot_sync(0xffffffffu, bf));
    }
  }
  if (lane == 0) {
    RowStat st; st.m = m; st.s = s; st.arg = arg; st.pad = before;
    w.stats[(size_t)tile * R + r] = st;
  }
}

// ---------------------------------------------------------------------------------------------
// a10 tail + a11..a15: merge statistics, judge scores, acceptance bits, first rejection, next
// token (greedy), new cache length and commit.  One block per sequence.
// ---------------------------------------------------------------------------------------------
__global__ void k_finalize(const StepArgs* __restrict__ args, KvView kv, Work w, Dims dm, int n_vtiles, int R) {
  pdl_wait();
  pdl_launch();
  __shared__ RowStat sred[256];
  __shared__ RowStat rs[kMaxGamma + 1];
  __shared__ float score[kMaxGamma + 1];
  const int b = blockIdx.x, gamma = args->gamma, rows = gamma + 1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = blockDim.x >> 5;
  const int seq = args->seq_ids[b];
  // merged statistics of every row: thread t folds tiles t, t+T, ... in order, then a fixed tree
  for (int j = 0; j < rows; ++j) {
    const int r = b * rows + j;
    RowStat a; a.m = -INFINITY; a.s = 0.f; a.arg = 0; a.pad = 0;
    // contiguous ranges keep vocabulary order inside and across threads
    int per = (n_vtiles + blockDim.x - 1) / blockDim.x;
    int t0 = tid * per, t1 = min(t0 + per, n_vtiles);
    for (int t = t0; t < t1; ++t) a = stat_merge(a, w.stats[(size_t)t * R + r]);
    sred[tid] = a;
    __syncthreads();
    for (int stride = 1; stride < (int)blockDim.x; stride <<= 1) {
      if ((tid % (2 * stride)) == 0 && tid + stride < (int)blockDim.x) sred[tid] = stat_merge(sred[tid], sred[tid + stride]);
      __syncthreads();
    }
    if (tid == 0) { rs[j] = sred[0]; w.rowstat[r] = sred[0]; }
    __syncthreads();
  }
  // judge scores: Verifier(h_j) = sigmoid(w.h_j + b), j = 1..gamma, one warp per row
  for (int j = 1 + warp; j <= gamma; j += nwarp) {
    const float* h = w.Hf + (size_t)(b * rows + j) * dm.d;
    float a = 0.f;
    if (args->has_judge)
      for (int i = lane; i < dm.d; i += 32) a = fmaf(h[i], w.judge_w[i], a);
    a = warp_sum(a);
    if (lane == 0) {
      float s = args->has_judge ? 1.0f / (1.0f + expf(-(a + args->judge_bias))) : 0.f;
      score[j] = s;
      args->judge_scores[b * gamma + j - 1] = s;
    }
  }
  __syncthreads();
  if (warp == 0) {
    bool ok = true;  // lanes >= gamma do not constrain the scan
    if (lane < gamma) {
      const int j = lane + 1;  // drafted position
      const int d = args->draft_ids[b * gamma + lane];
      const RowStat st = rs[j - 1];
      const float zd = w.tgt_logit[b * rows + j - 1] - st.m;
      const float p = expf(zd) / st.s;
      args->p_draft[b * gamma + lane] = p;
      if (args->logp_draft) args->logp_draft[b * gamma + lane] = zd - logf(st.s);
      bool align;
      if (args->mode == 0) align = args->top_k >= 2 ? st.pad < args->top_k : (d == st.arg);
      else align = args->uniforms[b * rows + lane] * args->q_tok[b * gamma + lane] < p;
      bool judge = args->has_judge && (score[j] > args->theta[b]);
      ok = (args->use_align && align) || (args->use_judge && judge) || args->accept_all;
    }
    unsigned rej = __ballot_sync(0xffffffffu, !ok);
    int n = rej ? (__ffs(rej) - 1) : gamma;
    if (lane == 0) {
      const int L = w.row_pos[b * rows];
      args->accepted_len[b] = n;
      args->new_kv_len[b] = L + 1 + n;
      if (args->mode == 0) {
        int nxt = rs[n].arg;
        args->next_token[b] = nxt;
        if (args->commit) kv.pending[seq] = nxt;
      }
      if (args->commit) kv.kv_len[seq] = L + 1 + n;
    }
  }
}

// a14, sampling mode, first half: the row the emitted token is drawn from (row n_b of sequence b, known only
// after the first-rejection scan) is normalised again into a compact set of GEMM input planes, one row per
// sequence; a second LM-head pass over those B rows then yields the only logits the step ever stores.
template <typename T>
__global__ void k_select_rows(const StepArgs* __restrict__ args, Work w, Dims dm, const T* __restrict__ gain) {
  extern __shared__ float xs[];
  __shared__ float red[32];
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x, rows = args->gamma + 1;
  const int r = b * rows + min(max(args->accepted_len[b], 0), rows - 1);
  for (int i = threadIdx.x; i < dm.d; i += blockDim.x) xs[i] = w.X[(size_t)r * dm.d + i];
  __syncthreads();
  norm_row_from_smem<T>(xs, dm.d, gain, dm.eps, w.Asel, gridDim.x, b, nullptr, nullptr, red);
}

// a14, sampling mode: inverse CDF over the vocabulary of norm(max(0, p_n - q_{n+1})) (first
// rejection) or of p_gamma (everything accepted), driven by uniforms[:, gamma].  fp64 prefix sums.
// per_seq: the logit scratch holds one row per sequence (row b) instead of every block row.
__global__ void k_resample(const StepArgs* __restrict__ args, KvView kv, Work w, Dims dm, int per_seq) {
  pdl_wait();
  pdl_launch();
  __shared__ double part[1024];
  __shared__ double total_s;
  __shared__ int winner;
  const int b = blockIdx.x, gamma = args->gamma, rows = gamma + 1, tid = threadIdx.x, T = blockDim.x;
  const int n = args->accepted_len[b];
  const int r = b * rows + n;
  const RowStat st = w.rowstat[r];
  const float invT = args->inv_temperature;
  const float* lg = w.logits + (size_t)(per_seq ? b : r) * dm.V;
  const float* q = (n < gamma) ? args->q_full + ((size_t)b * gamma + n) * dm.V : nullptr;
  const int per = (dm.V + T - 1) / T, v0 = tid * per, v1 = min(v0 + per, dm.V);
  const double inv_s = 1.0 / (double)st.s;
  for (int pass = 0; pass < 2; ++pass) {
    const bool residual = (q != nullptr) && pass == 0;
    double acc = 0.0;
    for (int v = v0; v < v1; ++v) {
      double p = (double)expf(lg[v] * invT - st.m) * inv_s;
      acc += residual ? fmax(0.0, p - (double)q[v]) : p;
    }
    part[tid] = acc;
    __syncthreads();
    if (tid == 0) {
      double run = 0.0;
      for (int i = 0; i < T; ++i) { double t = part[i]; part[i] = run; run += t; }  // exclusive prefix
      total_s = run;
      winner = dm.V - 1;
    }
    __syncthreads();
    const double total = total_s;
    if (residual && !(total > 0.0)) { __syncthreads(); continue; }  // no residual mass: fall back to p
    const double target = (double)args->uniforms[b * rows + gamma] * total;
    double run = part[tid];
    for (int v = v0; v < v1; ++v) {
      double p = (double)expf(lg[v] * invT - st.m) * inv_s;
      run += residual ? fmax(0.0, p - (double)q[v]) : p;
      if (run > target) { atomicMin(&winner, v); break; }
    }
    __syncthreads();
    if (tid == 0) {
      args->next_token[b] = winner;
      if (args->commit) kv.pending[args->seq_ids[b]] = winner;
    }
    break;
  }
}

// Rollback: kv_len <- new_len where new_len <= kv_len, else flag the error and leave it.
__global__ void k_rollback(KvView kv, const int* __restrict__ seqs, const int* __restrict__ new_len, int B, int* status) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B) return;
  int s = seqs[i], n = new_len[i];
  if (n >= 0 && n <= kv.kv_len[s]) kv.kv_len[s] = n;
  else atomicCAS(status, DEV_OK, DEV_STATE);
}

// Copy rows between a contiguous [n, Hkv, hd] buffer and the paged pool (fill: to_pool = 1).
template <typename T>
__global__ void k_kv_copy(KvView kv, int seq, int layer, int start, int n_tokens, T* k, T* v, int to_pool) {
  const int t = blockIdx.x;
  if (t >= n_tokens) return;
  const int pos = start + t;
  const int page = kv.block_table[(size_t)seq * kv.max_pages_per_seq + pos / kv.page_size];
  const int slot = pos % kv.page_size;
  const int width = kv.n_kv_heads * kv.head_dim;
  for (int i = threadIdx.x; i < width; i += blockDim.x) {
    int h = i / kv.head_dim, dd = i % kv.head_dim;
    T* kr = kv_row<T>(kv, layer, page, 0, h, slot) + dd;
    T* vr = kv_row<T>(kv, layer, page, 1, h, slot) + dd;
    if (to_pool) { *kr = k[(size_t)t * width + i]; *vr = v[(size_t)t * width + i]; }
    else { k[(size_t)t * width + i] = *kr; v[(size_t)t * width + i] = *vr; }
  }
}

}  // namespace sj
