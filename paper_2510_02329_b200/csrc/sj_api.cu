// Host runtime and C ABI of the verification step: handles, paged-KV bookkeeping, argument checks,
// launch sequence (optionally replayed as a CUDA graph with programmatic dependent launches).
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <tuple>
#include <vector>

#include "../../include/sj.h"
#include "sj_attn_tc.cuh"
#include "sj_attn_t5.cuh"
#include "sj_gemm_tc.cuh"
#include "sj_mega.cuh"

using namespace sj;

// ---------------------------------------------------------------------------------------------
// errors
// ---------------------------------------------------------------------------------------------
static thread_local char g_err[512] = "";

static sj_status fail(sj_status st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return st;
}

#define CU_TRY(expr)                                                                              \
  do {                                                                                            \
    cudaError_t e_ = (expr);                                                                      \
    if (e_ != cudaSuccess) {                                                                      \
      cudaGetLastError();                                                                         \
      return fail(e_ == cudaErrorMemoryAllocation ? SJ_ERR_OOM : SJ_ERR_CUDA, "%s: %s", #expr,    \
                  cudaGetErrorString(e_));                                                        \
    }                                                                                             \
  } while (0)

extern "C" const char* sj_last_error(void) { return g_err; }

// Every device allocation and release of the library goes through these two, so that a caller (or a test)
// can check that a call it believes allocation-free really is (sj_device_memory_calls()).
static std::atomic<long> g_mem_calls{0};
static cudaError_t counted_malloc(void** p, size_t bytes) {
  g_mem_calls.fetch_add(1, std::memory_order_relaxed);
  return cudaMalloc(p, bytes);
}
static cudaError_t counted_free(void* p) {
  g_mem_calls.fetch_add(1, std::memory_order_relaxed);
  return cudaFree(p);
}
extern "C" long sj_device_memory_calls(void) { return g_mem_calls.load(std::memory_order_relaxed); }

// ---------------------------------------------------------------------------------------------
// launch helper (programmatic dependent launch attribute on request)
// ---------------------------------------------------------------------------------------------
template <typename... KArgs, typename... Args>
static cudaError_t launch(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                          Args&&... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(std::forward<Args>(args))...);
}

// ---------------------------------------------------------------------------------------------
// TMA descriptors (driver entry point fetched at run time: no link-time dependency on libcuda)
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

static sj_status get_encode() {
  if (g_encode) return SJ_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  CU_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (!fn || qres != cudaDriverEntryPointSuccess) return fail(SJ_ERR_CUDA, "cuTensorMapEncodeTiled not available");
  g_encode = (EncodeTiledFn)fn;
  return SJ_OK;
}

// bf16 row-major [rows, K] matrix, box = [box_rows, 64] with 128-byte swizzle, zero fill out of bounds
static sj_status make_map(CUtensorMap* tm, const void* base, long rows, long K, int box_rows) {
  sj_status st = get_encode();
  if (st != SJ_OK) return st;
  if ((reinterpret_cast<uintptr_t>(base) & 15) != 0 || (K * 2) % 16 != 0)
    return fail(SJ_ERR_INVALID_ARG, "bf16 matrix must be 16-byte aligned with K a multiple of 8");
  cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t gstr[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstr, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(SJ_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
  return SJ_OK;
}

// ---------------------------------------------------------------------------------------------
// tensor-core GEMM sites
// ---------------------------------------------------------------------------------------------
struct TcSite {
  // static per site
  int N = 0, K = 0, n_tiles = 0, KB = 0, G = 0, nseg = 0;
  int seg_tile_end[3] = {0, 0, 0};
  int max_slots = 1;
  int2* d_tile_slots = nullptr;
  bool lm = false;
};

static int round_up(int x, int m) { return (x + m - 1) / m * m; }

// Which blocks contribute to which tile (must mirror the kernel's u_lo/u_hi arithmetic).
static void build_tile_slots(int n_tiles, int KB, int G, std::vector<int2>& out, int& max_slots) {
  long long U = (long long)n_tiles * KB;
  out.assign(n_tiles, make_int2(0, 0));
  std::vector<int> first(n_tiles, -1), cnt(n_tiles, 0);
  for (int c = 0; c < G; ++c) {
    long long lo = (long long)c * U / G, hi = (long long)(c + 1) * U / G;
    if (hi <= lo) continue;
    int t0 = (int)(lo / KB), t1 = (int)((hi - 1) / KB);
    for (int t = t0; t <= t1; ++t) {
      if (first[t] < 0) first[t] = c;
      cnt[t] = c - first[t] + 1;
    }
  }
  max_slots = 1;
  for (int t = 0; t < n_tiles; ++t) {
    out[t] = make_int2(first[t], cnt[t]);
    max_slots = std::max(max_slots, cnt[t]);
  }
}

struct RowGeom {  // how R activation rows are fed to the MMA
  int NB, nblk, a_blocks, plane_rows, acc_stride, acc_bufs, stages, a_stage_bytes;
  uint32_t tmem_cols;
  size_t smem_bytes;
};

// `merged`: R counts the rows of ONE plane; the stage holds both planes and the lo plane's products are
// accumulated into the hi plane's columns.
static RowGeom row_geom(int R, bool merged = false) {
  RowGeom g;
  int rp = round_up(std::max(R, 1), 16);
  g.NB = rp > 256 ? 2 : 1;
  g.nblk = round_up((rp + g.NB - 1) / g.NB, 16);
  int cols = g.NB * g.nblk;
  g.acc_bufs = (2 * cols <= 512) ? 2 : 1;
  g.acc_stride = cols;
  uint32_t need = (uint32_t)(cols * g.acc_bufs), tc = 32;
  while (tc < need) tc <<= 1;
  g.tmem_cols = tc;
  g.a_blocks = merged ? 2 * g.NB : g.NB;
  g.plane_rows = merged ? rp : 0;
  g.a_stage_bytes = round_up((merged ? 2 : 1) * cols * 128, 1024);
  int stage = kWTileBytes + g.a_stage_bytes;
  const int budget = 200 * 1024;
  g.stages = std::max(2, std::min(12, budget / stage));
  g.smem_bytes = (size_t)g.stages * stage + sizeof(TcSmemCtl) + 1024;
  return g;
}

// ---------------------------------------------------------------------------------------------
// handles
// ---------------------------------------------------------------------------------------------
struct LayerW {
  const void *wq, *wk, *wv, *wo, *wg, *wu, *wd, *na, *nf, *bq, *bk, *bv;
  CUtensorMap m_q, m_k, m_v, m_o, m_g, m_u, m_d;
  CUtensorMap m_g64, m_u64;   // gate / up with boxes of 64 rows (whole-step kernel)
};

struct StepKey {
  int B, gamma, mode, chunk_len, gemm_impl, attn_impl, pdl, scratch;
  bool operator<(const StepKey& o) const {
    return std::tie(B, gamma, mode, chunk_len, gemm_impl, attn_impl, pdl, scratch) <
           std::tie(o.B, o.gamma, o.mode, o.chunk_len, o.gemm_impl, o.attn_impl, o.pdl, o.scratch);
  }
};

struct sj_target {
  sj_model_config cfg;
  Dims dm;
  cudaStream_t stream = nullptr;
  int device = 0, sm_count = 0, max_rows = 64;
  bool bf = false;
  const void *embed = nullptr, *lm_head = nullptr, *final_norm = nullptr;
  CUtensorMap m_lm;
  std::vector<LayerW> layers;
  Work work;
  StepArgs* d_args = nullptr;
  float* d_judge_w = nullptr;
  int* d_prefill = nullptr;        // device scratch of sj_prefill(): one block's token ids and outputs
  double* d_inv_freq = nullptr;
  float theta = 0.5f, judge_bias = 0.f;
  bool has_judge = false;
  int opt_gemm = 0, opt_attn = 0, opt_graph = 1, opt_pdl = 1, opt_timing = 0, opt_step = 0, opt_trace = 0, opt_ring = 0, opt_att_precise = 1, opt_a5_min_tiles = 4;
  bool mega_shapes = false, coop = false;
  MegaLayerPtrs* d_layer_ptrs = nullptr;
  float* d_sumsq = nullptr;
  unsigned* d_sync = nullptr;      // [0] barrier counter, [1] abort word, [2..3] timeout note; [64 ..) the split-K
                                   // partial words (64-bit, [blocks][Rp][128]); zeroed as one range before every launch
  unsigned long long* d_trace = nullptr;
  std::vector<MegaMaps> mega_maps;  // one per launch chunk of kMegaMaxLayers layers
  struct Timed { const char* name; cudaEvent_t a, b; };
  std::vector<Timed> timed;
  TcSite s_qkv, s_o, s_gu, s_down, s_lm;
  size_t p_elems = 0;
  size_t att_chunks_cap = 0;
  int att_rows_cap = 0;
  size_t tc_part_cap = 0;   // floats in tc_m / tc_l
  size_t logits_rows = 0;
  std::map<StepKey, cudaGraphExec_t> graphs;
  std::map<int, CUtensorMap> mapA_d, mapA_q, mapA_f, mapA_sel;  // activation maps per R (mapA_sel: per B)
  std::vector<void*> owned;
};

struct sj_kv {
  sj_target* t = nullptr;
  KvView view;
  int max_seqs = 0;
  long max_pages = 0;
  std::vector<std::vector<int>> pages;  // per sequence
  std::vector<int> free_pages;
  std::vector<int> len_hi;              // upper bound of the live length known to the host
  std::vector<char> exact;              // len_hi is the exact length
  int* d_block_table = nullptr;
  int* d_tmp = nullptr;                 // [2 * SJ_MAX_BATCH] staging for rollback / set_len
  CUtensorMap tm_pool;                  // bf16 pool as a [rows, head_dim] matrix, box = 16 slots x 64 dims
  bool has_tm_pool = false;
};

static void clear_graphs(sj_target* t) {
  for (auto& kvp : t->graphs) cudaGraphExecDestroy(kvp.second);
  t->graphs.clear();
}

template <typename T>
static sj_status dev_alloc(sj_target* t, T** p, size_t n) {
  void* q = nullptr;
  cudaError_t e = counted_malloc(&q, std::max<size_t>(n, 1) * sizeof(T));
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(e == cudaErrorMemoryAllocation ? SJ_ERR_OOM : SJ_ERR_CUDA, "cudaMalloc(%zu bytes): %s", n * sizeof(T),
                cudaGetErrorString(e));
  }
  *p = reinterpret_cast<T*>(q);
  if (t) t->owned.push_back(q);
  return SJ_OK;
}

static sj_status setup_site(sj_target* t, TcSite& s, int nseg, const int* seg_rows, int K, bool lm) {
  s.nseg = nseg;
  s.K = K;
  s.KB = K / kBK;
  s.lm = lm;
  int tiles = 0;
  s.N = 0;
  for (int i = 0; i < 3; ++i) {
    if (i < nseg) {
      tiles += (seg_rows[i] + kTileN - 1) / kTileN;
      s.N += seg_rows[i];
    }
    s.seg_tile_end[i] = tiles;
  }
  s.n_tiles = tiles;
  s.G = std::min(t->sm_count, lm ? tiles : (int)std::min<long long>((long long)tiles * s.KB, t->sm_count));
  if (!lm) {
    std::vector<int2> slots;
    build_tile_slots(tiles, s.KB, s.G, slots, s.max_slots);
    sj_status st = dev_alloc(t, &s.d_tile_slots, slots.size());
    if (st != SJ_OK) return st;
    CU_TRY(cudaMemcpy(s.d_tile_slots, slots.data(), slots.size() * sizeof(int2), cudaMemcpyHostToDevice));
  }
  return SJ_OK;
}

static bool tc_shapes_ok(const sj_model_config& c) {
  auto m128 = [](int x) { return x % 128 == 0; };
  return c.dtype == SJ_DTYPE_BF16 && m128(c.n_q_heads * c.head_dim) && m128(c.n_kv_heads * c.head_dim) &&
         m128(c.d_ffn) && m128(c.d_model) && c.d_model % kBK == 0 && c.d_ffn % kBK == 0 &&
         (c.n_q_heads * c.head_dim) % kBK == 0;
}

typedef void (*MegaKernel)(const MegaMaps, const MegaParams, const StepArgs*, const KvView, const Work, const Dims);
// The persistent kernel for a head dimension (64 or 128), a number of row slots (4, 6 or 8), with or without
// the timeline code, with the mma.sync or (head dimension 128 only) the tcgen05 attention phase.
template <bool TR, bool A5>
static MegaKernel mega_kernel_t(int hd, int ns) {
  if (hd == 128)
    return ns == 4 ? k_verify_mega<128, 4, TR, A5> : (ns == 6 ? k_verify_mega<128, 6, TR, A5> : k_verify_mega<128, 8, TR, A5>);
  return ns == 4 ? k_verify_mega<64, 4, TR, false> : (ns == 6 ? k_verify_mega<64, 6, TR, false> : k_verify_mega<64, 8, TR, false>);
}
static MegaKernel mega_kernel(int hd, int ns, bool trace, bool a5) {
  if (a5) return trace ? mega_kernel_t<true, true>(hd, ns) : mega_kernel_t<false, true>(hd, ns);
  return trace ? mega_kernel_t<true, false>(hd, ns) : mega_kernel_t<false, false>(hd, ns);
}

extern "C" sj_status sj_create_target(const sj_model_config* cfg, const sj_weights* w, void* cuda_stream,
                                      sj_target** out) {
  if (!cfg || !w || !out) return fail(SJ_ERR_INVALID_ARG, "null argument");
  *out = nullptr;
  const sj_model_config& c = *cfg;
  if (c.n_layers <= 0 || c.d_model <= 0 || c.n_q_heads <= 0 || c.n_kv_heads <= 0 || c.head_dim <= 0 ||
      c.d_ffn <= 0 || c.vocab <= 0)
    return fail(SJ_ERR_INVALID_ARG, "non-positive dimension");
  if (c.dtype != SJ_DTYPE_F32 && c.dtype != SJ_DTYPE_BF16) return fail(SJ_ERR_INVALID_ARG, "unknown dtype %d", c.dtype);
  if (c.head_dim != 64 && c.head_dim != 128) return fail(SJ_ERR_SHAPE, "head_dim must be 64 or 128");
  if (c.n_q_heads % c.n_kv_heads != 0) return fail(SJ_ERR_SHAPE, "n_q_heads must be a multiple of n_kv_heads");
  if (c.d_model % 8 || c.d_ffn % 8) return fail(SJ_ERR_SHAPE, "d_model and d_ffn must be multiples of 8");
  if (c.d_model > 12288) return fail(SJ_ERR_SHAPE, "d_model above 12288 is not supported");
  if (!(c.rms_eps >= 0.f) || !(c.rope_theta > 0.f)) return fail(SJ_ERR_INVALID_ARG, "bad rms_eps / rope_theta");
  int max_rows = c.max_rows > 0 ? c.max_rows : 64;
  if (max_rows > SJ_MAX_ROWS) return fail(SJ_ERR_SHAPE, "max_rows above %d", SJ_MAX_ROWS);
  if (!w->embed || !w->lm_head || !w->final_norm || !w->wq || !w->wk || !w->wv || !w->wo || !w->w_gate || !w->w_up ||
      !w->w_down || !w->norm_attn || !w->norm_ffn)
    return fail(SJ_ERR_INVALID_ARG, "null weight pointer");
  if (c.qkv_bias && (!w->bq || !w->bk || !w->bv)) return fail(SJ_ERR_INVALID_ARG, "qkv_bias set but biases missing");
  for (int l = 0; l < c.n_layers; ++l) {
    if (!w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->w_gate[l] || !w->w_up[l] || !w->w_down[l] ||
        !w->norm_attn[l] || !w->norm_ffn[l])
      return fail(SJ_ERR_INVALID_ARG, "null weight pointer in layer %d", l);
    if (c.qkv_bias && (!w->bq[l] || !w->bk[l] || !w->bv[l])) return fail(SJ_ERR_INVALID_ARG, "null bias in layer %d", l);
  }
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  CU_TRY(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return fail(SJ_ERR_UNSUPPORTED, "built for sm_100a; device is sm_%d%d", prop.major, prop.minor);

  sj_target* t = new sj_target();
  t->cfg = c;
  t->dm = Dims{c.n_layers, c.d_model, c.n_q_heads, c.n_kv_heads, c.head_dim, c.d_ffn, c.vocab, c.rms_eps};
  t->stream = (cudaStream_t)cuda_stream;
  t->device = dev;
  t->sm_count = prop.multiProcessorCount;
  t->max_rows = max_rows;
  t->bf = c.dtype == SJ_DTYPE_BF16;
  t->embed = w->embed;
  t->lm_head = w->lm_head;
  t->final_norm = w->final_norm;
  t->layers.resize(c.n_layers);
  for (int l = 0; l < c.n_layers; ++l) {
    LayerW& L = t->layers[l];
    L.wq = w->wq[l]; L.wk = w->wk[l]; L.wv = w->wv[l]; L.wo = w->wo[l];
    L.wg = w->w_gate[l]; L.wu = w->w_up[l]; L.wd = w->w_down[l];
    L.na = w->norm_attn[l]; L.nf = w->norm_ffn[l];
    L.bq = c.qkv_bias ? w->bq[l] : nullptr; L.bk = c.qkv_bias ? w->bk[l] : nullptr; L.bv = c.qkv_bias ? w->bv[l] : nullptr;
  }
  const bool tc = tc_shapes_ok(c);
  t->opt_gemm = tc ? 1 : 0;
  t->opt_attn = t->bf ? (c.head_dim == 128 ? 2 : 1) : 0;
  t->opt_graph = t->stream ? 1 : 0;  // the legacy default stream cannot be captured

  sj_status st = SJ_OK;
  auto bail = [&](sj_status s) { sj_destroy_target(t); return s; };
  const size_t esz = t->bf ? 2 : 4;
  const int qd = c.n_q_heads * c.head_dim, kd = c.n_kv_heads * c.head_dim, R = max_rows;
  Work& W = t->work;
  memset(&W, 0, sizeof(W));
  uint8_t* tmp = nullptr;
#define ALLOC(field, type, count)                                                     \
  do {                                                                                \
    type* p_ = nullptr;                                                               \
    if ((st = dev_alloc(t, &p_, (count))) != SJ_OK) return bail(st);                  \
    field = p_;                                                                       \
  } while (0)
  ALLOC(W.X, float, (size_t)R * c.d_model);
  const size_t act_rows = t->bf ? (size_t)2 * pad16(R) : (size_t)R;  // bf16: hi and lo planes
  ALLOC(tmp, uint8_t, act_rows * c.d_model * esz); W.A = tmp;
  ALLOC(W.Q, float, (size_t)R * qd);
  if (t->bf) ALLOC(W.Qb, __half, (size_t)R * qd);
  if (t->bf) ALLOC(W.Qlo, __half, (size_t)R * qd);
  if (t->bf) ALLOC(W.KVn, __half, (size_t)R * 2 * kd);
  ALLOC(tmp, uint8_t, act_rows * qd * esz); W.ATT = tmp;
  ALLOC(tmp, uint8_t, act_rows * c.d_ffn * esz); W.H = tmp;
  ALLOC(tmp, uint8_t, act_rows * c.d_model * esz); W.Asel = tmp;   // at most one row per sequence is used
  ALLOC(W.Hf, float, (size_t)R * c.d_model);
  ALLOC(W.rope, float2, (size_t)R * (c.head_dim / 2));
  ALLOC(W.row_pos, int, R);
  ALLOC(W.chunk_start, int, SJ_MAX_BATCH + 1);
  const int n_vtiles = (c.vocab + kTileN - 1) / kTileN;
  ALLOC(W.stats, RowStat, (size_t)n_vtiles * R);
  ALLOC(W.tgt_logit, float, R);
  ALLOC(W.tgt_pre, float, R);
  ALLOC(W.rowstat, RowStat, R);
  ALLOC(W.status, int, 1);
  ALLOC(t->d_args, StepArgs, 1);
  ALLOC(t->d_judge_w, float, c.d_model);
  ALLOC(t->d_inv_freq, double, c.head_dim / 2);
  W.judge_w = t->d_judge_w;
  W.inv_freq = t->d_inv_freq;
  {
    cudaError_t e = cudaMemset(W.status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(t->d_judge_w, 0, sizeof(float) * c.d_model);
    if (e == cudaSuccess) e = cudaMemset(W.tgt_logit, 0, sizeof(float) * R);
    std::vector<double> inv(c.head_dim / 2);
    for (int i = 0; i < c.head_dim / 2; ++i) inv[i] = std::pow((double)c.rope_theta, -2.0 * i / c.head_dim);
    if (e == cudaSuccess) e = cudaMemcpy(t->d_inv_freq, inv.data(), inv.size() * sizeof(double), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { fail(SJ_ERR_CUDA, "workspace init: %s", cudaGetErrorString(e)); return bail(SJ_ERR_CUDA); }
  }
  // GEMM sites and the partial buffer
  size_t p_elems = (size_t)R * std::max({qd + 2 * kd, c.d_model, 2 * c.d_ffn});
  if (tc) {
    int seg_qkv[3] = {qd, kd, kd}, seg_o[1] = {c.d_model}, seg_gu[2] = {c.d_ffn, c.d_ffn}, seg_d[1] = {c.d_model},
        seg_lm[1] = {c.vocab};
    if ((st = setup_site(t, t->s_qkv, 3, seg_qkv, c.d_model, false)) != SJ_OK) return bail(st);
    if ((st = setup_site(t, t->s_o, 1, seg_o, qd, false)) != SJ_OK) return bail(st);
    if ((st = setup_site(t, t->s_gu, 2, seg_gu, c.d_model, false)) != SJ_OK) return bail(st);
    if ((st = setup_site(t, t->s_down, 1, seg_d, c.d_ffn, false)) != SJ_OK) return bail(st);
    if ((st = setup_site(t, t->s_lm, 1, seg_lm, c.d_model, true)) != SJ_OK) return bail(st);
    p_elems = 0;
    for (TcSite* s : {&t->s_qkv, &t->s_o, &t->s_gu, &t->s_down})
      p_elems = std::max(p_elems, (size_t)s->max_slots * R * s->N);
    for (int l = 0; l < c.n_layers; ++l) {
      LayerW& L = t->layers[l];
      if ((st = make_map(&L.m_q, L.wq, qd, c.d_model, kTileN)) != SJ_OK) return bail(st);
      if ((st = make_map(&L.m_k, L.wk, kd, c.d_model, kTileN)) != SJ_OK) return bail(st);
      if ((st = make_map(&L.m_v, L.wv, kd, c.d_model, kTileN)) != SJ_OK) return bail(st);
      if ((st = make_map(&L.m_o, L.wo, c.d_model, qd, kTileN)) != SJ_OK) return bail(st);
      if ((st = make_map(&L.m_g, L.wg, c.d_ffn, c.d_model, kTileN)) != SJ_OK) return bail(st);
      if ((st = make_map(&L.m_u, L.wu, c.d_ffn, c.d_model, kTileN)) != SJ_OK) return bail(st);
      if ((st = make_map(&L.m_d, L.wd, c.d_model, c.d_ffn, kTileN)) != SJ_OK) return bail(st);
      if ((st = make_map(&L.m_g64, L.wg, c.d_ffn, c.d_model, 64)) != SJ_OK) return bail(st);
      if ((st = make_map(&L.m_u64, L.wu, c.d_ffn, c.d_model, 64)) != SJ_OK) return bail(st);
    }
    if ((st = make_map(&t->m_lm, t->lm_head, c.vocab, c.d_model, kTileN)) != SJ_OK) return bail(st);
    cudaError_t e = cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) { fail(SJ_ERR_CUDA, "smem opt-in: %s", cudaGetErrorString(e)); return bail(SJ_ERR_CUDA); }
  }
  t->p_elems = p_elems;
  ALLOC(W.P, float, p_elems);
  {
    int coop = 0;
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    t->coop = coop != 0;
  }
  t->mega_shapes = tc && t->coop && c.d_ffn % 64 == 0;
  if (t->mega_shapes) {
    const int Rm = std::min(R, kMegaMaxRows);
    ALLOC(t->d_layer_ptrs, MegaLayerPtrs, c.n_layers);
    ALLOC(t->d_sumsq, float, (size_t)2 * (c.d_model / kTileN) * kMegaMaxRows);
    ALLOC(t->d_sync, unsigned, 64 + (size_t)4 * t->sm_count * pad16(Rm) * kTileN);
    std::vector<MegaLayerPtrs> lp(c.n_layers);
    for (int l = 0; l < c.n_layers; ++l) {
      const LayerW& L = t->layers[l];
      lp[l].bq = (const bf16*)L.bq; lp[l].bk = (const bf16*)L.bk; lp[l].bv = (const bf16*)L.bv;
      lp[l].gain_ffn = (const bf16*)L.nf;
      lp[l].gain_next = (const bf16*)(l + 1 < c.n_layers ? t->layers[l + 1].na : t->final_norm);
    }
    cudaError_t e = cudaMemcpy(t->d_layer_ptrs, lp.data(), lp.size() * sizeof(MegaLayerPtrs), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(t->d_sumsq, 0, sizeof(float) * 2 * (c.d_model / kTileN) * kMegaMaxRows);
    if (e == cudaSuccess) e = cudaMemset(t->d_sync, 0, sizeof(unsigned) * (64 + (size_t)4 * t->sm_count * pad16(Rm) * kTileN));
    for (int ns = 4; ns <= 8 && e == cudaSuccess; ns += 2)
      for (int v = 0; v < 4 && e == cudaSuccess; ++v)
        e = cudaFuncSetAttribute(mega_kernel(c.head_dim, ns, (v & 1) != 0, (v & 2) != 0 && c.head_dim == 128),
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) { fail(SJ_ERR_CUDA, "whole-step kernel set-up: %s", cudaGetErrorString(e)); return bail(SJ_ERR_CUDA); }
    for (int l0 = 0; l0 < c.n_layers; l0 += kMegaMaxLayers) {
      t->mega_maps.emplace_back();
      MegaMaps& mm = t->mega_maps.back();
      memset(&mm, 0, sizeof(mm));
      for (int l = l0; l < std::min(c.n_layers, l0 + kMegaMaxLayers); ++l) {
        const LayerW& L = t->layers[l];
        mm.wq[l - l0] = L.m_q; mm.wk[l - l0] = L.m_k; mm.wv[l - l0] = L.m_v; mm.wo[l - l0] = L.m_o;
        mm.wg[l - l0] = L.m_g64; mm.wu[l - l0] = L.m_u64; mm.wd[l - l0] = L.m_d;
      }
      mm.lm = t->m_lm;
    }
    // the activation planes are read as GEMM operands: rows past R must stay finite
    cudaMemset(W.A, 0, act_rows * c.d_model * esz);
    cudaMemset(W.ATT, 0, act_rows * qd * esz);
    cudaMemset(W.H, 0, act_rows * c.d_ffn * esz);
    cudaMemset(W.Asel, 0, act_rows * c.d_model * esz);
    t->opt_step = 1;
  }
#undef ALLOC
  if (t->bf && c.head_dim == 128) {
    cudaError_t e = cudaFuncSetAttribute(k_attn_t5, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kT5SmemBytes + sizeof(T5Ctl) + 1024));
    if (e != cudaSuccess) { fail(SJ_ERR_CUDA, "smem opt-in: %s", cudaGetErrorString(e)); return bail(SJ_ERR_CUDA); }
  }
  if (t->bf) {
    const int att_smem = kAttStages * kAttStageBytes + (int)sizeof(AttSmemCtl) + 1024;
    cudaError_t e = c.head_dim == 128
                        ? cudaFuncSetAttribute(k_attn_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, att_smem)
                        : cudaFuncSetAttribute(k_attn_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, att_smem);
    if (e != cudaSuccess) { fail(SJ_ERR_CUDA, "smem opt-in: %s", cudaGetErrorString(e)); return bail(SJ_ERR_CUDA); }
  }
  {
    cudaError_t e;
    if (t->bf) e = cudaFuncSetAttribute(k_attn_simt<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    else e = cudaFuncSetAttribute(k_attn_simt<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    if (e != cudaSuccess) { fail(SJ_ERR_CUDA, "smem opt-in: %s", cudaGetErrorString(e)); return bail(SJ_ERR_CUDA); }
  }
  *out = t;
  return SJ_OK;
}

extern "C" sj_status sj_destroy_target(sj_target* t) {
  if (!t) return SJ_OK;
  cudaStreamSynchronize(t->stream);
  clear_graphs(t);
  for (auto& e : t->timed) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
  for (void* p : t->owned) counted_free(p);
  delete t;
  cudaGetLastError();
  return SJ_OK;
}

extern "C" sj_status sj_load_judge_head(sj_target* t, const float* w_host, float bias, float theta) {
  if (!t || !w_host) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (!(theta == theta) || !(bias == bias)) return fail(SJ_ERR_INVALID_ARG, "NaN judge parameter");
  CU_TRY(cudaMemcpyAsync(t->d_judge_w, w_host, sizeof(float) * t->dm.d, cudaMemcpyHostToDevice, t->stream));
  CU_TRY(cudaStreamSynchronize(t->stream));
  t->judge_bias = bias;
  t->theta = theta;
  t->has_judge = true;
  return SJ_OK;
}

extern "C" sj_status sj_set_option(sj_target* t, const char* name, int value) {
  if (!t || !name) return fail(SJ_ERR_INVALID_ARG, "null argument");
  std::string n(name);
  if (n == "gemm_impl") {
    if (value != 0 && value != 1) return fail(SJ_ERR_INVALID_ARG, "gemm_impl must be 0 or 1");
    if (value == 1 && !tc_shapes_ok(t->cfg)) return fail(SJ_ERR_UNSUPPORTED, "tensor-core GEMM needs bf16 and 128-multiples");
    t->opt_gemm = value;
  } else if (n == "attn_impl") {
    if (value < 0 || value > 2) return fail(SJ_ERR_INVALID_ARG, "attn_impl must be 0, 1 or 2");
    if (value >= 1 && !t->bf) return fail(SJ_ERR_UNSUPPORTED, "tensor-core attention needs a bf16 model");
    if (value == 2 && t->dm.hd != 128) return fail(SJ_ERR_UNSUPPORTED, "the tcgen05 attention needs head_dim 128");
    t->opt_attn = value;
  } else if (n == "step_impl") {
    if (value != 0 && value != 1) return fail(SJ_ERR_INVALID_ARG, "step_impl must be 0 or 1");
    if (value == 1 && !t->mega_shapes) return fail(SJ_ERR_UNSUPPORTED, "the whole-step kernel needs bf16, 128-multiples and cooperative launch");
    t->opt_step = value;
  } else if (n == "ring_stages") {
    if (value != 0 && (value < 3 || value > kMegaMaxStages)) return fail(SJ_ERR_INVALID_ARG, "ring_stages must be 0 (auto) or 3..%d", kMegaMaxStages);
    t->opt_ring = value;
  } else if (n == "attn_tcgen05_min_tiles") {
    if (value < 0) return fail(SJ_ERR_INVALID_ARG, "attn_tcgen05_min_tiles must be >= 0");
    t->opt_a5_min_tiles = value;
  } else if (n == "attn_two_term_layers") {
    if (value < 0) return fail(SJ_ERR_INVALID_ARG, "attn_two_term_layers must be >= 0");
    cudaStreamSynchronize(t->stream);
    clear_graphs(t);
    t->opt_att_precise = value;
  } else if (n == "trace") {
    const size_t n_tr = kMegaTraceEntries;
    if (value && !t->d_trace) {
      sj_status st = dev_alloc(t, &t->d_trace, n_tr);
      if (st != SJ_OK) return st;
    }
    if (t->d_trace) CU_TRY(cudaMemsetAsync(t->d_trace, 0, sizeof(unsigned long long) * n_tr, t->stream));
    t->opt_trace = value > 0 ? value : 0;   // value k traces block k - 1
  } else if (n == "graph") {
    if (value && !t->stream) return fail(SJ_ERR_UNSUPPORTED, "the legacy default stream cannot be captured into a graph");
    t->opt_graph = value ? 1 : 0;
  } else if (n == "pdl") {
    t->opt_pdl = value ? 1 : 0;
  } else if (n == "timing") {
    cudaStreamSynchronize(t->stream);
    for (auto& e : t->timed) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
    t->timed.clear();
    t->opt_timing = value ? 1 : 0;
  } else {
    return fail(SJ_ERR_INVALID_ARG, "unknown option '%s'", name);
  }
  return SJ_OK;
}

extern "C" sj_status sj_sync(sj_target* t) {
  if (!t) return fail(SJ_ERR_INVALID_ARG, "null argument");
  int st = 0;
  CU_TRY(cudaMemcpyAsync(&st, t->work.status, sizeof(int), cudaMemcpyDeviceToHost, t->stream));
  CU_TRY(cudaStreamSynchronize(t->stream));
  if (st != 0) {
    CU_TRY(cudaMemsetAsync(t->work.status, 0, sizeof(int), t->stream));
    if (st == DEV_TIMEOUT && t->d_sync) {
      unsigned info[4] = {0, 0, 0, 0};   // the whole-step kernel notes which wait gave up first
      CU_TRY(cudaMemcpy(info, t->d_sync, sizeof(info), cudaMemcpyDeviceToHost));
      return fail(SJ_ERR_TIMEOUT, "a bounded device-side wait ran out (barrier count %u, wait kind %u in block %u, detail %u)",
                  info[0], info[2] & 255u, info[2] >> 8, info[3]);
    }
    return fail((sj_status)st, st == DEV_TIMEOUT ? "a bounded device-side wait ran out"
                                                 : "device rejected a state change (rollback beyond the live length)");
  }
  return SJ_OK;
}

// One block whose first thread runs one of the library's bounded waits on something that nothing will ever
// signal, with a small poll limit: the wait gives up, records DEV_TIMEOUT, and the kernel returns normally.
__global__ void k_expire_wait(int kind, uint32_t limit, unsigned* word, int* abort_g, int* status) {
  __shared__ uint64_t bar;
  __shared__ MegaCtl ctl;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    ctl.abort_flag = 0;
    if (kind == 0) {
      mbar_wait(smem_u32(&bar), 0, &ctl.abort_flag, status, limit);                      // stand-alone GEMM kernels
    } else if (kind == 1) {
      att_mbar_wait(smem_u32(&bar), 0, &ctl.abort_flag, status, abort_g, 15, 0, limit);  // ring / accumulator waits
    } else {
      MegaParams p;
      p.abort_g = abort_g;
      mega_spin_ge(word, 1u, &ctl, p, status, 15, 0, limit);                             // device-wide barrier poll
    }
  }
}

extern "C" sj_status sj_debug_expire_wait(sj_target* t, int kind, unsigned max_polls) {
  if (!t) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (kind < 0 || kind > 2) return fail(SJ_ERR_INVALID_ARG, "kind must be 0, 1 or 2");
  if (max_polls == 0 || max_polls > (1u << 20)) return fail(SJ_ERR_INVALID_ARG, "max_polls must be in [1, 2^20]");
  if (!t->d_sync) return fail(SJ_ERR_UNSUPPORTED, "this target has no whole-step kernel workspace");
  // [1] abort word, [2..3] timeout note (as in a step), [8] the word that stays zero
  CU_TRY(cudaMemsetAsync(t->d_sync, 0, sizeof(unsigned) * 16, t->stream));
  CU_TRY(launch(k_expire_wait, dim3(1), dim3(32), 0, t->stream, false, kind, (uint32_t)max_polls, t->d_sync + 8,
                reinterpret_cast<int*>(t->d_sync + 1), t->work.status));
  return SJ_OK;
}

// ---------------------------------------------------------------------------------------------
// KV cache
// ---------------------------------------------------------------------------------------------
extern "C" sj_status sj_kv_create(sj_target* t, int max_seqs, long max_pages, int page_size, sj_kv** out) {
  if (!t || !out) return fail(SJ_ERR_INVALID_ARG, "null argument");
  *out = nullptr;
  if (page_size != 16) return fail(SJ_ERR_UNSUPPORTED, "page_size must be 16");
  if (max_seqs <= 0 || max_pages <= 0 || max_pages > 0x7fffffffL) return fail(SJ_ERR_INVALID_ARG, "bad max_seqs/max_pages");
  sj_kv* kv = new sj_kv();
  kv->t = t;
  kv->max_seqs = max_seqs;
  kv->max_pages = max_pages;
  const size_t esz = t->bf ? 2 : 4;
  const size_t page_elems = (size_t)2 * t->dm.Hkv * page_size * t->dm.hd;
  const size_t bytes = (size_t)t->dm.n_layers * max_pages * page_elems * esz;
  void* pool = nullptr;
  cudaError_t e = counted_malloc(&pool, bytes);
  int* meta = nullptr;
  const int mpps = (int)std::min<long>(max_pages, 1 << 20);
  if (e == cudaSuccess) e = counted_malloc((void**)&meta, sizeof(int) * ((size_t)max_seqs * (mpps + 2) + 2 * SJ_MAX_BATCH));
  if (e != cudaSuccess) {
    cudaGetLastError();
    if (pool) counted_free(pool);
    delete kv;
    return fail(e == cudaErrorMemoryAllocation ? SJ_ERR_OOM : SJ_ERR_CUDA, "KV pool of %zu bytes: %s", bytes,
                cudaGetErrorString(e));
  }
  cudaMemset(meta, 0, sizeof(int) * ((size_t)max_seqs * (mpps + 2) + 2 * SJ_MAX_BATCH));
  // Slots past a sequence's length are read (and masked) by the tensor-core attention: keep them finite.
  e = cudaMemset(pool, 0, bytes);
  if (e == cudaSuccess && t->bf) {
    const long long rows_total = (long long)t->dm.n_layers * max_pages * 2 * t->dm.Hkv * page_size;
    if (rows_total < 0x7fffffffLL && make_map(&kv->tm_pool, pool, rows_total, t->dm.hd, page_size) == SJ_OK)
      kv->has_tm_pool = true;
  }
  if (e != cudaSuccess) {
    cudaGetLastError();
    counted_free(pool);
    counted_free(meta);
    delete kv;
    return fail(SJ_ERR_CUDA, "KV pool clear: %s", cudaGetErrorString(e));
  }
  kv->d_block_table = meta;
  kv->view.pool = pool;
  kv->view.block_table = meta;
  kv->view.kv_len = meta + (size_t)max_seqs * mpps;
  kv->view.pending = kv->view.kv_len + max_seqs;
  kv->d_tmp = kv->view.pending + max_seqs;
  kv->view.n_pages = max_pages;
  kv->view.max_pages_per_seq = mpps;
  kv->view.page_size = page_size;
  kv->view.n_kv_heads = t->dm.Hkv;
  kv->view.head_dim = t->dm.hd;
  kv->pages.resize(max_seqs);
  kv->len_hi.assign(max_seqs, 0);
  kv->exact.assign(max_seqs, 1);
  kv->free_pages.resize(max_pages);
  for (long i = 0; i < max_pages; ++i) kv->free_pages[i] = (int)(max_pages - 1 - i);  // pop_back yields 0,1,2..
  *out = kv;
  return SJ_OK;
}

extern "C" sj_status sj_kv_destroy(sj_kv* kv) {
  if (!kv) return SJ_OK;
  cudaStreamSynchronize(kv->t->stream);
  clear_graphs(kv->t);  // captured steps hold this cache's pointers
  counted_free(kv->view.pool);
  counted_free(kv->d_block_table);
  delete kv;
  cudaGetLastError();
  return SJ_OK;
}

// Make sure `seq` owns pages for `tokens` tokens; uploads the new block-table entries.
static sj_status reserve(sj_kv* kv, int seq, long tokens, std::vector<std::pair<int, int>>* undo) {
  const int ps = kv->view.page_size;
  const long need = (tokens + ps - 1) / ps;
  std::vector<int>& pg = kv->pages[seq];
  if (need > kv->view.max_pages_per_seq) return fail(SJ_ERR_OOM, "sequence %d would exceed the block table", seq);
  const size_t had = pg.size();
  if ((long)had >= need) return SJ_OK;
  if ((long)kv->free_pages.size() < need - (long)had)
    return fail(SJ_ERR_OOM, "KV page pool exhausted (%zu free, %ld needed)", kv->free_pages.size(), need - (long)had);
  while ((long)pg.size() < need) {
    pg.push_back(kv->free_pages.back());
    kv->free_pages.pop_back();
  }
  if (undo) undo->push_back({seq, (int)had});
  CU_TRY(cudaMemcpyAsync(kv->d_block_table + (size_t)seq * kv->view.max_pages_per_seq + had, pg.data() + had,
                         sizeof(int) * (pg.size() - had), cudaMemcpyHostToDevice, kv->t->stream));
  return SJ_OK;
}

static void release_beyond(sj_kv* kv, int seq, long tokens) {
  const int ps = kv->view.page_size;
  const size_t keep = (size_t)((tokens + ps - 1) / ps);
  std::vector<int>& pg = kv->pages[seq];
  while (pg.size() > keep) {
    kv->free_pages.push_back(pg.back());
    pg.pop_back();
  }
}

static sj_status check_seqs(sj_kv* kv, const int* seq_ids, int B) {
  if (!kv || !seq_ids) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (B <= 0 || B > SJ_MAX_BATCH) return fail(SJ_ERR_INVALID_ARG, "B out of range");
  for (int i = 0; i < B; ++i)
    if (seq_ids[i] < 0 || seq_ids[i] >= kv->max_seqs) return fail(SJ_ERR_INVALID_ARG, "sequence id %d out of range", seq_ids[i]);
  return SJ_OK;
}

extern "C" sj_status sj_kv_fill(sj_kv* kv, int seq, int layer, int start, int n_tokens, const void* k, const void* v) {
  if (!kv || !k || !v) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (seq < 0 || seq >= kv->max_seqs || layer < 0 || layer >= kv->t->dm.n_layers || start < 0 || n_tokens <= 0)
    return fail(SJ_ERR_INVALID_ARG, "sj_kv_fill: index out of range");
  sj_status st = reserve(kv, seq, (long)start + n_tokens, nullptr);
  if (st != SJ_OK) return st;
  cudaError_t e;
  if (kv->t->bf)
    e = launch(k_kv_copy<bf16>, dim3(n_tokens), dim3(256), 0, kv->t->stream, false, kv->view, seq, layer, start, n_tokens,
               (bf16*)k, (bf16*)v, 1);
  else
    e = launch(k_kv_copy<float>, dim3(n_tokens), dim3(256), 0, kv->t->stream, false, kv->view, seq, layer, start, n_tokens,
               (float*)k, (float*)v, 1);
  CU_TRY(e);
  return SJ_OK;
}

extern "C" sj_status sj_kv_read(sj_kv* kv, int seq, int layer, int start, int n_tokens, void* k_out, void* v_out) {
  if (!kv || !k_out || !v_out) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (seq < 0 || seq >= kv->max_seqs || layer < 0 || layer >= kv->t->dm.n_layers || start < 0 || n_tokens <= 0)
    return fail(SJ_ERR_INVALID_ARG, "sj_kv_read: index out of range");
  if ((size_t)(start + n_tokens) > kv->pages[seq].size() * kv->view.page_size)
    return fail(SJ_ERR_INVALID_ARG, "sj_kv_read: rows beyond the reserved pages");
  cudaError_t e;
  if (kv->t->bf)
    e = launch(k_kv_copy<bf16>, dim3(n_tokens), dim3(256), 0, kv->t->stream, false, kv->view, seq, layer, start, n_tokens,
               (bf16*)k_out, (bf16*)v_out, 0);
  else
    e = launch(k_kv_copy<float>, dim3(n_tokens), dim3(256), 0, kv->t->stream, false, kv->view, seq, layer, start, n_tokens,
               (float*)k_out, (float*)v_out, 0);
  CU_TRY(e);
  CU_TRY(cudaStreamSynchronize(kv->t->stream));
  return SJ_OK;
}

extern "C" sj_status sj_kv_set_len(sj_kv* kv, const int* seq_ids, const int* lens, int B) {
  sj_status st = check_seqs(kv, seq_ids, B);
  if (st != SJ_OK) return st;
  if (!lens) return fail(SJ_ERR_INVALID_ARG, "null argument");
  for (int i = 0; i < B; ++i)
    if (lens[i] < 0 || (size_t)lens[i] > kv->pages[seq_ids[i]].size() * kv->view.page_size)
      return fail(SJ_ERR_STATE, "length %d of sequence %d exceeds its reserved rows", lens[i], seq_ids[i]);
  for (int i = 0; i < B; ++i) {
    CU_TRY(cudaMemcpyAsync(kv->view.kv_len + seq_ids[i], lens + i, sizeof(int), cudaMemcpyHostToDevice, kv->t->stream));
    kv->len_hi[seq_ids[i]] = lens[i];
    kv->exact[seq_ids[i]] = 1;
  }
  return SJ_OK;
}

extern "C" sj_status sj_kv_set_pending(sj_kv* kv, const int* seq_ids, const int* tokens, int B) {
  sj_status st = check_seqs(kv, seq_ids, B);
  if (st != SJ_OK) return st;
  if (!tokens) return fail(SJ_ERR_INVALID_ARG, "null argument");
  for (int i = 0; i < B; ++i) {
    if (tokens[i] < 0 || tokens[i] >= kv->t->dm.V) return fail(SJ_ERR_INVALID_ARG, "token id out of range");
  }
  for (int i = 0; i < B; ++i)
    CU_TRY(cudaMemcpyAsync(kv->view.pending + seq_ids[i], tokens + i, sizeof(int), cudaMemcpyHostToDevice, kv->t->stream));
  return SJ_OK;
}

extern "C" sj_status sj_kv_len(sj_kv* kv, const int* seq_ids, int* out_len, int B) {
  sj_status st = check_seqs(kv, seq_ids, B);
  if (st != SJ_OK) return st;
  if (!out_len) return fail(SJ_ERR_INVALID_ARG, "null argument");
  for (int i = 0; i < B; ++i)
    CU_TRY(cudaMemcpyAsync(out_len + i, kv->view.kv_len + seq_ids[i], sizeof(int), cudaMemcpyDeviceToHost, kv->t->stream));
  CU_TRY(cudaStreamSynchronize(kv->t->stream));
  for (int i = 0; i < B; ++i) {
    kv->len_hi[seq_ids[i]] = out_len[i];
    kv->exact[seq_ids[i]] = 1;
    release_beyond(kv, seq_ids[i], out_len[i]);
  }
  return SJ_OK;
}

extern "C" sj_status sj_rollback_kv(sj_kv* kv, const int* seq_ids, const int* new_len, int B) {
  sj_status st = check_seqs(kv, seq_ids, B);
  if (st != SJ_OK) return st;
  if (!new_len) return fail(SJ_ERR_INVALID_ARG, "null argument");
  for (int i = 0; i < B; ++i) {
    if (new_len[i] < 0) return fail(SJ_ERR_INVALID_ARG, "negative length");
    if (new_len[i] > kv->len_hi[seq_ids[i]])
      return fail(SJ_ERR_STATE, "rollback of sequence %d to %d beyond its length (at most %d)", seq_ids[i], new_len[i],
                  kv->len_hi[seq_ids[i]]);
  }
  int stage[2 * SJ_MAX_BATCH];
  memcpy(stage, seq_ids, sizeof(int) * B);
  memcpy(stage + B, new_len, sizeof(int) * B);
  CU_TRY(cudaMemcpyAsync(kv->d_tmp, stage, sizeof(int) * 2 * B, cudaMemcpyHostToDevice, kv->t->stream));
  CU_TRY(launch(k_rollback, dim3((B + 127) / 128), dim3(128), 0, kv->t->stream, false, kv->view, (const int*)kv->d_tmp,
                (const int*)(kv->d_tmp + B), B, kv->t->work.status));
  // Whole pages past the new length go back to the pool.  Everything that still touches them (a verify in
  // flight, this rollback) was enqueued on the target's stream before any later call can hand them out
  // again, and that call's kernels run on the same stream.  If the device refuses the rollback (the live
  // length turned out shorter than new_len) the pages kept for new_len still cover it.
  for (int i = 0; i < B; ++i) {
    kv->len_hi[seq_ids[i]] = new_len[i];
    release_beyond(kv, seq_ids[i], new_len[i]);
  }
  return SJ_OK;
}

// ---------------------------------------------------------------------------------------------
// the step
// ---------------------------------------------------------------------------------------------
// How R activation rows reach the MMA.  Two bf16 planes (hi at row 0, lo at row pad16(R)): as 2 * pad16(R)
// accumulator columns that the epilogue adds, while those fit the 512 TMEM columns; beyond that (R > 256)
// the lo plane's products are accumulated into the hi plane's columns by a second MMA per K step.
static bool planes_fit(int R) { return 2 * pad16(R) <= 512; }
static RowGeom feed_geom(int R, bool planes) {
  if (!planes) return row_geom(R);
  return planes_fit(R) ? row_geom(2 * pad16(R)) : row_geom(pad16(R), true);
}

static sj_status activation_map(sj_target* t, std::map<int, CUtensorMap>& cache, const void* base, int R, int K,
                                const CUtensorMap** out) {
  auto it = cache.find(R);
  if (it == cache.end()) {
    CUtensorMap m;
    RowGeom g = feed_geom(R, true);
    sj_status st = make_map(&m, base, 2 * pad16(R), K, g.nblk);
    if (st != SJ_OK) return st;
    it = cache.emplace(R, m).first;
  }
  *out = &it->second;
  return SJ_OK;
}

static cudaError_t launch_tc(sj_target* t, const TcSite& s, const CUtensorMap* mA, const CUtensorMap* w0,
                             const CUtensorMap* w1, const CUtensorMap* w2, int R, bool pdl, bool planes, int lm_mode = -1,
                             const Work* work = nullptr) {
  RowGeom g = feed_geom(R, planes);
  TcGemmParams p;
  memset(&p, 0, sizeof(p));
  p.lo_off = (planes && planes_fit(R)) ? pad16(R) : 0;
  p.a_blocks = g.a_blocks; p.plane_rows = g.plane_rows;
  p.n_tiles = s.n_tiles; p.KB = s.KB; p.G = s.G; p.U = (long long)s.n_tiles * s.KB; p.R = R;
  p.NB = g.NB; p.nblk = g.nblk; p.N_total = s.N;
  for (int i = 0; i < 3; ++i) p.seg_tile_end[i] = s.seg_tile_end[i];
  p.stages = g.stages; p.a_stage_bytes = g.a_stage_bytes; p.tmem_cols = g.tmem_cols;
  p.acc_bufs = g.acc_bufs; p.acc_stride = g.acc_stride;
  p.P = t->work.P; p.slot_stride = (size_t)R * s.N; p.tile_slots = s.d_tile_slots;
  p.lm_mode = lm_mode >= 0 ? lm_mode : (s.lm ? 1 : 0); p.status = t->work.status;
  return launch(k_gemm_tc, dim3(s.G), dim3(kTcThreads), g.smem_bytes, t->stream, pdl, *mA, *w0, *(w1 ? w1 : w0),
                *(w2 ? w2 : w0), p, (const StepArgs*)t->d_args, work ? *work : t->work, t->dm.V);
}

// a14 in sampling mode with the tensor-core LM head: re-normalise the one row per sequence that the emitted
// token is drawn from, run the LM head over those B rows into the [B, V] logit scratch, draw the token.
template <typename T>
static sj_status enqueue_resample(sj_target* t, sj_kv* kv, int B, const Work& W, bool pdl) {
  const Dims& dm = t->dm;
  cudaStream_t s = t->stream;
  const CUtensorMap* mA = nullptr;
  sj_status st = activation_map(t, t->mapA_sel, W.Asel, B, dm.d, &mA);
  if (st != SJ_OK) return st;
  CU_TRY(launch(k_select_rows<T>, dim3(B), dim3(256), sizeof(float) * dm.d, s, pdl, (const StepArgs*)t->d_args, W, dm,
                (const T*)t->final_norm));
  CU_TRY(launch_tc(t, t->s_lm, mA, &t->m_lm, nullptr, nullptr, B, pdl, true, 2, &W));
  CU_TRY(launch(k_resample, dim3(B), dim3(1024), 0, s, pdl, (const StepArgs*)t->d_args, kv->view, W, dm, 1));
  return SJ_OK;
}

template <typename T>
static cudaError_t launch_simt(sj_target* t, const void* A, const GemmSegs& segs, float* Y, int R, int N, int K, bool pdl) {
  return launch(k_gemm_simt<T, 8>, dim3((N + 7) / 8), dim3(256), 0, t->stream, pdl, (const T*)A, segs, Y, R, N, K,
                t->bf ? 2 : 1);
}

// Launch `expr`; in timing mode bracket it with events filed under `name`.
#define TIMED(name, expr)                                                        \
  do {                                                                           \
    cudaEvent_t ea_ = nullptr, eb_ = nullptr;                                    \
    if (timing) {                                                                \
      CU_TRY(cudaEventCreate(&ea_));                                             \
      CU_TRY(cudaEventCreate(&eb_));                                             \
      CU_TRY(cudaEventRecord(ea_, s));                                           \
    }                                                                            \
    CU_TRY(expr);                                                                \
    if (timing) {                                                                \
      CU_TRY(cudaEventRecord(eb_, s));                                           \
      t->timed.push_back({name, ea_, eb_});                                      \
    }                                                                            \
  } while (0)

template <typename T>
static sj_status enqueue_step(sj_target* t, sj_kv* kv, int B, int gamma, int mode, int chunk_len, bool use_scratch,
                               size_t n_chunks_hi) {
  const Dims& dm = t->dm;
  const int R = B * (gamma + 1), qd = dm.Hq * dm.hd, kd = dm.Hkv * dm.hd;
  const bool timing = t->opt_timing != 0 && !t->opt_graph;
  const bool pdl = t->opt_pdl != 0 && !timing, tc = t->opt_gemm == 1;
  const bool attn_tc = t->opt_attn >= 1 && t->bf && kv->has_tm_pool;
  const StepArgs* args = t->d_args;
  Work W = t->work;
  if (!use_scratch) W.logits = nullptr;
  if (!attn_tc) W.Qb = nullptr, W.KVn = nullptr;
  cudaStream_t s = t->stream;
  const size_t row_smem = sizeof(float) * dm.d;
  SplitPlan one{nullptr, 0};
  const CUtensorMap *mA_d = nullptr, *mA_q = nullptr, *mA_f = nullptr;
  if (tc) {
    sj_status st;
    if ((st = activation_map(t, t->mapA_d, W.A, R, dm.d, &mA_d)) != SJ_OK) return st;
    if ((st = activation_map(t, t->mapA_q, W.ATT, R, qd, &mA_q)) != SJ_OK) return st;
    if ((st = activation_map(t, t->mapA_f, W.H, R, dm.F, &mA_f)) != SJ_OK) return st;
  }
  auto plan_of = [&](const TcSite& site) { return tc ? SplitPlan{site.d_tile_slots, site.n_tiles} : one; };

  TIMED("plan", launch(k_plan, dim3(1), dim3(256), 0, s, false, args, kv->view, W, chunk_len));
  TIMED("embed_norm", launch(k_embed_norm<T>, dim3(R), dim3(256), row_smem, s, pdl, args, kv->view, W, dm, (const T*)t->embed,
                (const T*)t->layers[0].na));
  const int nq = (dm.Hq / dm.Hkv) * (gamma + 1);
  const size_t att_smem = sizeof(float) * ((size_t)nq * dm.hd + kAttKT * (dm.hd + 1) + kAttKT * dm.hd + (size_t)nq * kAttKT + 3 * nq);
  const int att_grid = std::max(1, std::min<int>(t->sm_count * 2, (int)n_chunks_hi * dm.Hkv));
  for (int l = 0; l < dm.n_layers; ++l) {
    const LayerW& L = t->layers[l];
    // QKV projection
    if (tc) {
      TIMED("gemm_qkv", launch_tc(t, t->s_qkv, mA_d, &L.m_q, &L.m_k, &L.m_v, R, pdl, true));
    } else {
      GemmSegs g{{L.wq, L.wk, L.wv}, {qd, kd, kd}, 3};
      TIMED("gemm_cudacore", launch_simt<T>(t, W.A, g, W.P, R, qd + 2 * kd, dm.d, pdl));
    }
    TIMED("qkv_rope", launch(k_qkv_rope<T>, dim3(R), dim3(256), 0, s, pdl, args, kv->view, W, dm, plan_of(t->s_qkv),
                  (size_t)R * (qd + 2 * kd), l, (const T*)L.bq, (const T*)L.bk, (const T*)L.bv));
    // attention
    if (attn_tc) {
      AttArgs aa{W.Qb, l < t->opt_att_precise ? W.Qlo : nullptr, W.KVn, AttPartials{W.tc_m, W.tc_l, W.tc_o}, t->sm_count + B * dm.Hkv, l};
      const size_t tc_smem = kAttStages * kAttStageBytes + sizeof(AttSmemCtl) + 1024;
      const AttPartials parts{W.tc_m, W.tc_l, W.tc_o};
      // one warp per (sequence, KV head, query row, half of the head dimension): every task's loads are in flight at once
      const int items = B * dm.Hkv * nq, cgrid = std::max(1, std::min(32 * t->sm_count, (items * (dm.hd >= 128 ? 2 : 1) + 7) / 8));
      if (dm.hd == 128 && t->opt_attn == 2 && nq <= 128) {   // one 128-lane accumulator holds a KV head's query rows
        const size_t t5_smem = kT5SmemBytes + sizeof(T5Ctl) + 1024;
        TIMED("attn", launch(k_attn_t5, dim3(t->sm_count), dim3(kT5Threads), t5_smem, s, pdl, kv->tm_pool, args, kv->view, W, dm, aa));
        TIMED("attn_combine", launch(k_attn_combine_tc<128, 8>, dim3(cgrid), dim3(256), 0, s, pdl, args, W, dm, parts, t->sm_count, aa.n_tail_base, kT5Keys, kT5Pad));
      } else if (dm.hd == 128) {
        TIMED("attn", launch(k_attn_tc<128>, dim3(t->sm_count), dim3(kAttTcThreads), tc_smem, s, pdl, kv->tm_pool, args, kv->view, W, dm, aa));
        TIMED("attn_combine", launch(k_attn_combine_tc<128, 0>, dim3(cgrid), dim3(256), 0, s, pdl, args, W, dm, parts, t->sm_count, aa.n_tail_base, 0, 0));
      } else {
        TIMED("attn", launch(k_attn_tc<64>, dim3(t->sm_count), dim3(kAttTcThreads), tc_smem, s, pdl, kv->tm_pool, args, kv->view, W, dm, aa));
        TIMED("attn_combine", launch(k_attn_combine_tc<64, 0>, dim3(cgrid), dim3(256), 0, s, pdl, args, W, dm, parts, t->sm_count, aa.n_tail_base, 0, 0));
      }
    } else {
      TIMED("attn", launch(k_attn_simt<T>, dim3(att_grid), dim3(kAttThreads), att_smem, s, pdl, args, kv->view, W, dm, l, chunk_len));
      TIMED("attn_combine", launch(k_attn_combine<T>, dim3(R * dm.Hq), dim3(std::min(dm.hd, 128)), 0, s, pdl, args, W, dm));
    }
    // O projection + residual + FFN norm
    if (tc) {
      TIMED("gemm_o", launch_tc(t, t->s_o, mA_q, &L.m_o, nullptr, nullptr, R, pdl, true));
    } else {
      GemmSegs g{{L.wo, nullptr, nullptr}, {dm.d, 0, 0}, 1};
      TIMED("gemm_cudacore", launch_simt<T>(t, W.ATT, g, W.P, R, dm.d, qd, pdl));
    }
    TIMED("reduce_norm", launch(k_reduce_norm<T>, dim3(R), dim3(256), row_smem, s, pdl, args, W, dm, plan_of(t->s_o), (size_t)R * dm.d,
                  (const T*)L.nf, 0));
    // gate/up + SwiGLU
    if (tc) {
      TIMED("gemm_gateup", launch_tc(t, t->s_gu, mA_d, &L.m_g, &L.m_u, nullptr, R, pdl, true));
    } else {
      GemmSegs g{{L.wg, L.wu, nullptr}, {dm.F, dm.F, 0}, 2};
      TIMED("gemm_cudacore", launch_simt<T>(t, W.A, g, W.P, R, 2 * dm.F, dm.d, pdl));
    }
    TIMED("swiglu", launch(k_swiglu<T>, dim3((dm.F + 255) / 256, R), dim3(256), 0, s, pdl, W, dm, plan_of(t->s_gu),
                  (size_t)R * 2 * dm.F));
    // down projection + residual + next norm
    if (tc) {
      TIMED("gemm_down", launch_tc(t, t->s_down, mA_f, &L.m_d, nullptr, nullptr, R, pdl, true));
    } else {
      GemmSegs g{{L.wd, nullptr, nullptr}, {dm.d, 0, 0}, 1};
      TIMED("gemm_cudacore", launch_simt<T>(t, W.H, g, W.P, R, dm.d, dm.F, pdl));
    }
    const bool last = (l == dm.n_layers - 1);
    const void* gain = last ? t->final_norm : t->layers[l + 1].na;
    TIMED("reduce_norm", launch(k_reduce_norm<T>, dim3(R), dim3(256), row_smem, s, pdl, args, W, dm, plan_of(t->s_down),
                  (size_t)R * dm.d, (const T*)gain, last ? 1 : 0));
  }
  // LM head + statistics
  const int n_vtiles = (dm.V + kTileN - 1) / kTileN;
  if (tc) {
    TIMED("target_logits", launch(k_target_logits, dim3((R + 7) / 8), dim3(256), 0, s, pdl, args, W, dm, (const bf16*)t->lm_head, R));
    TIMED("gemm_lm_head", launch_tc(t, t->s_lm, mA_d, &t->m_lm, nullptr, nullptr, R, pdl, true, -1, &W));   // W: no [R, V] logit store
  } else {
    GemmSegs g{{t->lm_head, nullptr, nullptr}, {dm.V, 0, 0}, 1};
    TIMED("gemm_cudacore", launch_simt<T>(t, W.A, g, W.logits, R, dm.V, dm.d, pdl));
    TIMED("lm_stats", launch(k_lm_stats_from_logits, dim3(n_vtiles, (R + 7) / 8), dim3(256), 0, s, pdl, args, W, dm, R));
  }
  TIMED("finalize", launch(k_finalize, dim3(B), dim3(256), 0, s, pdl, args, kv->view, W, dm, n_vtiles, R));
  if (mode == SJ_MODE_SAMPLING) {
    if (tc) {
      sj_status st = enqueue_resample<T>(t, kv, B, t->work, pdl);   // t->work: with the [B, V] logit scratch
      if (st != SJ_OK) return st;
    } else {
      TIMED("resample", launch(k_resample, dim3(B), dim3(1024), 0, s, pdl, args, kv->view, W, dm, 0));
    }
  }
  return SJ_OK;
}

#undef TIMED

// The whole step as one cooperative launch per chunk of kMegaMaxLayers layers.
static bool mega_usable(const sj_target* t, const sj_kv* kv, int B, int gamma) {
  const int rows = gamma + 1, R = B * rows, group = t->dm.Hq / t->dm.Hkv;
  return t->opt_step == 1 && t->opt_gemm == 1 && t->mega_shapes && kv->has_tm_pool && R <= kMegaMaxRows &&
         group * rows <= 16 * 6 && t->stream != nullptr;
}

static sj_status launch_mega(sj_target* t, sj_kv* kv, int B, int gamma, int mode, bool use_scratch, long total_keys) {
  const Dims& dm = t->dm;
  const int rows = gamma + 1, R = B * rows, Rp = pad16(R), qd = dm.Hq * dm.hd;
  cudaStream_t s = t->stream;
  Work W = t->work;
  if (!use_scratch) W.logits = nullptr;
  const CUtensorMap *mA_d = nullptr, *mA_q = nullptr, *mA_f = nullptr;
  sj_status st;
  if ((st = activation_map(t, t->mapA_d, W.A, R, dm.d, &mA_d)) != SJ_OK) return st;
  if ((st = activation_map(t, t->mapA_q, W.ATT, R, qd, &mA_q)) != SJ_OK) return st;
  if ((st = activation_map(t, t->mapA_f, W.H, R, dm.F, &mA_f)) != SJ_OK) return st;
  MegaParams p;
  memset(&p, 0, sizeof(p));
  p.B = B; p.rows = rows; p.R = R; p.Rp = Rp;
  p.stage_bytes = kWTileBytes + round_up(2 * Rp * 128, 1024);
  // tcgen05 attention phase: head dimension 128, a KV head's query rows within two TMEM lane quarters, ring stages
  // that hold a 32 KiB key or value tile (49 block rows or more), and caches long enough that the phase is bound by
  // throughput (at a few tiles per block it is a chain of latencies, and the mma.sync phase, which needs no hand-over
  // between warps, is as fast)
  const int nq = (dm.Hq / dm.Hkv) * rows;
  const long tiles_per_block = total_keys * dm.Hkv / kA5Keys / t->sm_count;
  const bool a5 = dm.hd == 128 && nq <= kA5MaxRows && t->opt_attn == 2 && p.stage_bytes >= (int)kA5Part &&
                  tiles_per_block >= t->opt_a5_min_tiles;
  p.q_area_bytes = a5 ? a5_q_area_bytes(nq) : 0;
  const int ctl_bytes = ((int)sizeof(MegaCtl) + 127) & ~127;
  const int budget = 227 * 1024 - 1024 - ctl_bytes - p.q_area_bytes;
  p.stages = std::min(8, std::min(kMegaMaxStages, budget / p.stage_bytes));   // deeper rings did not measure faster; the rest stays L1
  if (p.stages < 3) return fail(SJ_ERR_SHAPE, "too many rows for the whole-step kernel");
  if (t->opt_ring) p.stages = std::min(p.stages, t->opt_ring);
  uint32_t tc = 32;
  while (tc < (uint32_t)(4 * Rp)) tc <<= 1;
  p.tmem_cols = a5 ? std::max(tc, (uint32_t)kA5TmemCols) : tc;
  p.lp = t->d_layer_ptrs;
  p.embed = (const bf16*)t->embed;
  p.lm_head = (const bf16*)t->lm_head;
  p.gain0 = (const bf16*)t->layers[0].na;
  p.sumsq = t->d_sumsq;
  p.pbuf = reinterpret_cast<unsigned long long*>(t->d_sync + 64);
  p.gbar = t->d_sync;
  p.abort_g = reinterpret_cast<int*>(t->d_sync + 1);
  p.n_tail_base = t->sm_count + B * dm.Hkv;
  p.att_precise_layers = t->opt_att_precise;
  p.trace = t->opt_trace ? t->d_trace : nullptr;
  p.trace_block = t->opt_trace ? (unsigned)std::min(t->opt_trace - 1, t->sm_count - 1) : 0u;
  const int grid = t->sm_count;
  const size_t smem = (size_t)p.stages * p.stage_bytes + p.q_area_bytes + ctl_bytes + 1024;
  const bool timing = t->opt_timing != 0;
  const int NL = dm.n_layers;
  for (size_t ci = 0; ci < t->mega_maps.size(); ++ci) {
    p.l0 = (int)ci * kMegaMaxLayers;
    p.l1 = std::min(NL, p.l0 + kMegaMaxLayers);
    p.do_embed = ci == 0 ? 1 : 0;
    p.do_lm = p.l1 == NL ? 1 : 0;
    MegaMaps mm = t->mega_maps[ci];
    mm.pool = kv->tm_pool;
    mm.a_d = *mA_d; mm.a_q = *mA_q; mm.a_f = *mA_f;
    CU_TRY(cudaMemsetAsync(t->d_sync, 0, sizeof(unsigned) * (64 + (size_t)4 * t->sm_count * Rp * kTileN), s));
    cudaEvent_t ea = nullptr, eb = nullptr;
    if (timing) {
      CU_TRY(cudaEventCreate(&ea));
      CU_TRY(cudaEventCreate(&eb));
      CU_TRY(cudaEventRecord(ea, s));
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kMegaThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    const StepArgs* args = t->d_args;
    // row slots per epilogue thread: a group gets at most (min(R, 16) + 1) / 2 rows of a 16-row chunk
    const int ns = R <= 8 ? 4 : (R <= 12 ? 6 : 8);
    CU_TRY(cudaLaunchKernelEx(&cfg, mega_kernel(dm.hd, ns, t->opt_trace != 0, a5), mm, p, args, kv->view, W, dm));
    if (timing) {
      CU_TRY(cudaEventRecord(eb, s));
      t->timed.push_back({"verify_step", ea, eb});
    }
  }
  if (mode == SJ_MODE_SAMPLING) return enqueue_resample<bf16>(t, kv, B, t->work, false);
  return SJ_OK;
}

extern "C" sj_status sj_step_trace(sj_target* t, unsigned long long* out_ns, int max_entries, int* n_entries) {
  if (!t || !out_ns || !n_entries || max_entries <= 0) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (!t->d_trace) return fail(SJ_ERR_STATE, "tracing was never enabled (sj_set_option \"trace\")");
  const int n = std::min(max_entries, kMegaTraceEntries);
  CU_TRY(cudaStreamSynchronize(t->stream));
  CU_TRY(cudaMemcpy(out_ns, t->d_trace, sizeof(unsigned long long) * n, cudaMemcpyDeviceToHost));
  *n_entries = n;
  return SJ_OK;
}

extern "C" sj_status sj_kernel_time(sj_target* t, const char* name, double* total_ms, long* launches) {
  if (!t || !name || !total_ms || !launches) return fail(SJ_ERR_INVALID_ARG, "null argument");
  CU_TRY(cudaStreamSynchronize(t->stream));
  double tot = 0.0;
  long n = 0;
  const size_t len = strlen(name);
  for (auto& e : t->timed) {
    if (strncmp(e.name, name, len) != 0) continue;  // prefix match: "gemm" covers every projection
    float ms = 0.f;
    CU_TRY(cudaEventElapsedTime(&ms, e.a, e.b));
    tot += ms;
    ++n;
  }
  *total_ms = tot;
  *launches = n;
  return SJ_OK;
}

static int pick_chunk_len(const sj_target* t, long total_keys) {
  long want = total_keys * t->dm.Hkv / (2L * t->sm_count);
  int ch = 64;
  while (ch < want && ch < 4096) ch <<= 1;
  return ch;
}

extern "C" sj_status sj_verify(sj_target* t, sj_kv* kv, const sj_verify_args* a, const sj_verify_out* o) {
  if (!t || !kv || !a || !o) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (kv->t != t) return fail(SJ_ERR_INVALID_ARG, "KV cache belongs to another target");
  if (a->B <= 0 || a->B > SJ_MAX_BATCH) return fail(SJ_ERR_INVALID_ARG, "B out of range");
  if (a->gamma < 1 || a->gamma > SJ_MAX_GAMMA) return fail(SJ_ERR_INVALID_ARG, "gamma out of range [1,%d]", SJ_MAX_GAMMA);
  const int B = a->B, gamma = a->gamma, rows = gamma + 1, R = B * rows;
  if (R > t->max_rows) return fail(SJ_ERR_SHAPE, "B*(gamma+1) = %d exceeds max_rows = %d", R, t->max_rows);
  sj_status st = check_seqs(kv, a->seq_ids, B);
  if (st != SJ_OK) return st;
  {
    std::vector<char> seen(kv->max_seqs, 0);
    for (int i = 0; i < B; ++i) {
      if (seen[a->seq_ids[i]]) return fail(SJ_ERR_INVALID_ARG, "duplicate sequence id %d", a->seq_ids[i]);
      seen[a->seq_ids[i]] = 1;
    }
  }
  if (a->mode != SJ_MODE_GREEDY && a->mode != SJ_MODE_SAMPLING) return fail(SJ_ERR_INVALID_ARG, "unknown mode");
  if (!a->draft_ids) return fail(SJ_ERR_INVALID_ARG, "draft_ids is null");
  if (a->mode == SJ_MODE_SAMPLING) {
    if (!a->draft_q_tok || !a->draft_q_full || !a->uniforms) return fail(SJ_ERR_INVALID_ARG, "sampling mode needs q and uniforms");
    if (!(a->temperature > 0.f)) return fail(SJ_ERR_INVALID_ARG, "temperature must be > 0");
  }
  if (!o->accepted_len || !o->next_token || !o->judge_scores || !o->p_draft || !o->new_kv_len)
    return fail(SJ_ERR_INVALID_ARG, "null output pointer");
  if (a->theta_override == a->theta_override && a->theta_override > 1e30f) return fail(SJ_ERR_INVALID_ARG, "bad theta");
  if (a->theta_override != a->theta_override) return fail(SJ_ERR_INVALID_ARG, "theta is NaN");
  if (a->theta_per_seq)
    for (int i = 0; i < a->B; ++i)
      if (!(a->theta_per_seq[i] >= 0.f && a->theta_per_seq[i] <= 1e30f)) return fail(SJ_ERR_INVALID_ARG, "theta_per_seq[%d] is not in [0, 1e30]", i);
  if (a->top_k < 0 || a->top_k > 2) return fail(SJ_ERR_UNSUPPORTED, "top_k must be 0, 1 or 2");
  if (a->top_k == 2 && a->mode != SJ_MODE_GREEDY) return fail(SJ_ERR_UNSUPPORTED, "top_k = 2 is a greedy-mode test");
  const int group = t->dm.Hq / t->dm.Hkv;
  if (group * rows > kAttMaxQ) return fail(SJ_ERR_SHAPE, "(Hq/Hkv)*(gamma+1) = %d exceeds %d", group * rows, kAttMaxQ);

  // a0: reserve pages for gamma+1 more rows per sequence; nothing is launched if the pool runs out
  std::vector<std::pair<int, int>> undo;
  long total_keys = 0;
  size_t chunk_need_base = 0;
  for (int i = 0; i < B; ++i) {
    int s = a->seq_ids[i];
    st = reserve(kv, s, (long)kv->len_hi[s] + rows, &undo);
    if (st != SJ_OK) {
      for (auto& u : undo) {
        std::vector<int>& pg = kv->pages[u.first];
        while ((int)pg.size() > u.second) { kv->free_pages.push_back(pg.back()); pg.pop_back(); }
      }
      return st;
    }
    total_keys += kv->len_hi[s] + rows;
  }
  const int chunk_len = pick_chunk_len(t, total_keys);
  for (int i = 0; i < B; ++i) chunk_need_base += (size_t)(kv->len_hi[a->seq_ids[i]] + rows + chunk_len - 1) / chunk_len;

  const bool use_mega = mega_usable(t, kv, B, gamma);
  // [R, V] logits exist only for the CUDA-core LM head (fp32 models, cross-checks); the tensor-core paths keep
  // softmax statistics per vocabulary tile and, in sampling mode, the logits of one row per sequence ([B, V])
  const bool use_scratch = t->opt_gemm == 0 && !use_mega;
  const size_t logit_rows_needed = use_scratch ? (size_t)R : (a->mode == SJ_MODE_SAMPLING ? (size_t)B : 0);
  // grow lazily-sized buffers (outside any capture)
  if (chunk_need_base > t->att_chunks_cap || rows > t->att_rows_cap) {
    CU_TRY(cudaStreamSynchronize(t->stream));
    clear_graphs(t);
    size_t cap = std::max(chunk_need_base * 2, (size_t)64);
    int rcap = std::max(rows, t->att_rows_cap);
    for (float** p : {&t->work.att_m, &t->work.att_l, &t->work.att_o}) {
      if (*p) {
        counted_free(*p);
        t->owned.erase(std::remove(t->owned.begin(), t->owned.end(), (void*)*p), t->owned.end());
        *p = nullptr;
      }
    }
    size_t n_ml = cap * t->dm.Hq * rcap;
    if ((st = dev_alloc(t, &t->work.att_m, n_ml)) != SJ_OK) return st;
    if ((st = dev_alloc(t, &t->work.att_l, n_ml)) != SJ_OK) return st;
    if ((st = dev_alloc(t, &t->work.att_o, n_ml * t->dm.hd)) != SJ_OK) return st;
    t->att_chunks_cap = cap;
    t->att_rows_cap = rcap;
  }
  if ((t->opt_attn >= 1 || use_mega) && t->bf && kv->has_tm_pool) {
    const size_t slots = (size_t)t->sm_count + 2 * (size_t)B * t->dm.Hkv;
    const size_t need = slots * kAttMaxSub * (size_t)(group * rows);
    if (need > t->tc_part_cap) {
      CU_TRY(cudaStreamSynchronize(t->stream));
      clear_graphs(t);
      for (float** p : {&t->work.tc_m, &t->work.tc_l, &t->work.tc_o}) {
        if (*p) {
          counted_free(*p);
          t->owned.erase(std::remove(t->owned.begin(), t->owned.end(), (void*)*p), t->owned.end());
          *p = nullptr;
        }
      }
      t->tc_part_cap = 0;
      if ((st = dev_alloc(t, &t->work.tc_m, need)) != SJ_OK) return st;
      if ((st = dev_alloc(t, &t->work.tc_l, need)) != SJ_OK) return st;
      if ((st = dev_alloc(t, &t->work.tc_o, need * t->dm.hd)) != SJ_OK) return st;
      // slots of blocks that own no tile are read with weight zero: they must hold finite values
      CU_TRY(cudaMemsetAsync(t->work.tc_m, 0, need * sizeof(float), t->stream));
      CU_TRY(cudaMemsetAsync(t->work.tc_l, 0, need * sizeof(float), t->stream));
      CU_TRY(cudaMemsetAsync(t->work.tc_o, 0, need * t->dm.hd * sizeof(float), t->stream));
      t->tc_part_cap = need;
    }
  }
  if (logit_rows_needed > t->logits_rows) {
    CU_TRY(cudaStreamSynchronize(t->stream));
    clear_graphs(t);
    if (t->work.logits) {
      counted_free(t->work.logits);
      t->owned.erase(std::remove(t->owned.begin(), t->owned.end(), (void*)t->work.logits), t->owned.end());
      t->work.logits = nullptr;
    }
    if ((st = dev_alloc(t, &t->work.logits, logit_rows_needed * t->dm.V)) != SJ_OK) return st;
    t->logits_rows = logit_rows_needed;
  }

  // per-call arguments: one small copy (the driver stages pageable memory before returning)
  StepArgs h;
  memset(&h, 0, sizeof(h));
  h.draft_ids = a->draft_ids; h.q_tok = a->draft_q_tok; h.q_full = a->draft_q_full; h.uniforms = a->uniforms;
  h.accepted_len = o->accepted_len; h.next_token = o->next_token; h.judge_scores = o->judge_scores;
  h.p_draft = o->p_draft; h.new_kv_len = o->new_kv_len; h.dbg_hidden = o->dbg_hidden; h.dbg_logits = o->dbg_logits;
  h.B = B; h.gamma = gamma; h.mode = a->mode; h.use_align = a->use_align ? 1 : 0; h.use_judge = a->use_judge ? 1 : 0;
  h.commit = a->commit ? 1 : 0;
  h.inv_temperature = a->mode == SJ_MODE_SAMPLING ? 1.0f / a->temperature : 1.0f;
  for (int i = 0; i < B; ++i)
    h.theta[i] = a->theta_per_seq ? a->theta_per_seq[i] : (a->theta_override >= 0.f ? a->theta_override : t->theta);
  h.top_k = a->top_k >= 2 ? 2 : 1;
  h.accept_all = a->accept_all ? 1 : 0;
  h.logp_draft = o->logp_draft;
  h.judge_bias = t->judge_bias;
  h.has_judge = t->has_judge ? 1 : 0;
  memcpy(h.seq_ids, a->seq_ids, sizeof(int) * B);
  CU_TRY(cudaMemcpyAsync(t->d_args, &h, sizeof(h), cudaMemcpyHostToDevice, t->stream));

  StepKey key{B, gamma, a->mode, chunk_len, t->opt_gemm, t->opt_attn, t->opt_pdl, use_scratch ? 1 : 0};
  if (use_mega) {
    if ((st = launch_mega(t, kv, B, gamma, a->mode, use_scratch, total_keys)) != SJ_OK) return st;
  } else if (t->opt_graph) {
    auto it = t->graphs.find(key);
    if (it == t->graphs.end()) {
      if (t->opt_gemm == 1) {  // encode activation maps before capturing
        const CUtensorMap* dummy;
        if ((st = activation_map(t, t->mapA_d, t->work.A, R, t->dm.d, &dummy)) != SJ_OK) return st;
      }
      cudaGraph_t graph = nullptr;
      CU_TRY(cudaStreamBeginCapture(t->stream, cudaStreamCaptureModeThreadLocal));
      st = t->bf ? enqueue_step<bf16>(t, kv, B, gamma, a->mode, chunk_len, use_scratch, chunk_need_base)
                 : enqueue_step<float>(t, kv, B, gamma, a->mode, chunk_len, use_scratch, chunk_need_base);
      cudaError_t e = cudaStreamEndCapture(t->stream, &graph);
      if (st != SJ_OK) {
        if (graph) cudaGraphDestroy(graph);
        cudaGetLastError();
        return st;
      }
      CU_TRY(e);
      cudaGraphExec_t exec = nullptr;
      e = cudaGraphInstantiate(&exec, graph, 0);
      cudaGraphDestroy(graph);
      CU_TRY(e);
      it = t->graphs.emplace(key, exec).first;
    }
    CU_TRY(cudaGraphLaunch(it->second, t->stream));
  } else {
    st = t->bf ? enqueue_step<bf16>(t, kv, B, gamma, a->mode, chunk_len, use_scratch, chunk_need_base)
               : enqueue_step<float>(t, kv, B, gamma, a->mode, chunk_len, use_scratch, chunk_need_base);
    if (st != SJ_OK) return st;
  }
  if (a->commit) {
    for (int i = 0; i < B; ++i) {
      int s = a->seq_ids[i];
      kv->len_hi[s] += rows;
      kv->exact[s] = 0;
    }
  }
  return SJ_OK;
}

// ---------------------------------------------------------------------------------------------
// chunked prefill and teacher-forced scoring: the verification step applied to known tokens
// ---------------------------------------------------------------------------------------------
// device scratch of one such block, in ints: [0,32) token ids, [32,64) accepted_len / next_token / new_kv_len,
// [64,96) judge scores, [96,128) p_draft, [128,160) and [160,192) log-probabilities of two blocks, [192,194) a score
constexpr int kBlockScratchInts = 8 * (SJ_MAX_GAMMA + 1);

// s = sum_k (lp_z[k] - lp_y[k]) in index order (fp64), s_prefix = lp_z[0] - lp_y[0]
__global__ void k_score_diff(const float* __restrict__ lp_z, const float* __restrict__ lp_y, int n, float* __restrict__ out) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    double s = 0.0;
    for (int k = 0; k < n; ++k) s += (double)lp_z[k] - (double)lp_y[k];
    out[0] = (float)s;
    out[1] = lp_z[0] - lp_y[0];
  }
}

extern "C" sj_status sj_semantic_score(sj_target* t, sj_kv* kv, int seq, int y_i, int z_i, const int* future, int n_future,
                                       float* score) {
  if (!t || !kv || !score || (n_future > 0 && !future)) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (kv->t != t) return fail(SJ_ERR_INVALID_ARG, "KV cache belongs to another target");
  if (seq < 0 || seq >= kv->max_seqs) return fail(SJ_ERR_INVALID_ARG, "sequence id %d out of range", seq);
  if (n_future < 0 || n_future + 1 > SJ_MAX_GAMMA) return fail(SJ_ERR_SHAPE, "n_future must be in [0, %d]", SJ_MAX_GAMMA - 1);
  for (int k = -2; k < n_future; ++k) {
    const int tok = k == -2 ? y_i : (k == -1 ? z_i : future[k]);
    if (tok < 0 || tok >= t->dm.V) return fail(SJ_ERR_INVALID_ARG, "token id out of range");
  }
  if (!t->d_prefill) {
    sj_status st = dev_alloc(t, &t->d_prefill, (size_t)kBlockScratchInts);
    if (st != SJ_OK) return st;
  }
  const int W = SJ_MAX_GAMMA + 1, gamma = n_future + 1;
  sj_verify_out o;
  memset(&o, 0, sizeof(o));
  o.accepted_len = t->d_prefill + W;
  o.next_token = o.accepted_len + 1;
  o.new_kv_len = o.accepted_len + 2;
  o.judge_scores = reinterpret_cast<float*>(t->d_prefill + 2 * W);
  o.p_draft = reinterpret_cast<float*>(t->d_prefill + 3 * W);
  float* lp[2] = {reinterpret_cast<float*>(t->d_prefill + 4 * W), reinterpret_cast<float*>(t->d_prefill + 5 * W)};
  float* d_score = reinterpret_cast<float*>(t->d_prefill + 6 * W);
  int block[SJ_MAX_GAMMA + 1];
  for (int k = 0; k < n_future; ++k) block[1 + k] = future[k];
  for (int pass = 0; pass < 2; ++pass) {   // the token-substituted response, then the original one
    block[0] = pass == 0 ? z_i : y_i;
    CU_TRY(cudaMemcpyAsync(t->d_prefill, block, sizeof(int) * gamma, cudaMemcpyHostToDevice, t->stream));
    sj_verify_args a;
    memset(&a, 0, sizeof(a));
    a.B = 1;
    a.gamma = gamma;
    a.seq_ids = &seq;
    a.draft_ids = t->d_prefill;
    a.mode = SJ_MODE_GREEDY;
    a.temperature = 1.f;
    a.theta_override = -1.f;
    a.accept_all = 1;
    a.commit = 0;          // the cache and the pending token stay as they are
    o.logp_draft = lp[pass];
    sj_status st = sj_verify(t, kv, &a, &o);
    if (st != SJ_OK) return st;
  }
  CU_TRY(launch(k_score_diff, dim3(1), dim3(32), 0, t->stream, false, (const float*)lp[0], (const float*)lp[1], gamma, d_score));
  CU_TRY(cudaMemcpyAsync(score, d_score, 2 * sizeof(float), cudaMemcpyDeviceToHost, t->stream));
  CU_TRY(cudaStreamSynchronize(t->stream));
  return SJ_OK;
}

extern "C" sj_status sj_prefill(sj_target* t, sj_kv* kv, int seq, const int* tokens, int n_tokens, int* next_token) {
  if (!t || !kv || !tokens) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (kv->t != t) return fail(SJ_ERR_INVALID_ARG, "KV cache belongs to another target");
  if (seq < 0 || seq >= kv->max_seqs) return fail(SJ_ERR_INVALID_ARG, "sequence id %d out of range", seq);
  if (n_tokens <= 0) return fail(SJ_ERR_INVALID_ARG, "n_tokens must be positive");
  for (int i = 0; i < n_tokens; ++i)
    if (tokens[i] < 0 || tokens[i] >= t->dm.V) return fail(SJ_ERR_INVALID_ARG, "token id out of range");
  const int group = t->dm.Hq / t->dm.Hkv;
  const int c_max = std::min({SJ_MAX_GAMMA + 1, kAttMaxQ / group, t->max_rows});
  if (c_max < 2) return fail(SJ_ERR_SHAPE, "max_rows = %d is too small for a prefill block", t->max_rows);
  if (!t->d_prefill) {   // draft ids and the step's outputs of one block
    sj_status st = dev_alloc(t, &t->d_prefill, (size_t)kBlockScratchInts);
    if (st != SJ_OK) return st;
  }
  int* d_draft = t->d_prefill;
  sj_verify_out o;
  memset(&o, 0, sizeof(o));
  o.accepted_len = t->d_prefill + (SJ_MAX_GAMMA + 1);
  o.next_token = o.accepted_len + 1;
  o.new_kv_len = o.accepted_len + 2;
  o.judge_scores = reinterpret_cast<float*>(t->d_prefill + 2 * (SJ_MAX_GAMMA + 1));
  o.p_draft = reinterpret_cast<float*>(t->d_prefill + 3 * (SJ_MAX_GAMMA + 1));
  for (int i = 0; i < n_tokens;) {
    const int c = std::min(c_max, n_tokens - i);
    sj_status st = sj_kv_set_pending(kv, &seq, tokens + i, 1);
    if (st != SJ_OK) return st;
    sj_verify_args a;
    memset(&a, 0, sizeof(a));
    a.B = 1;
    a.seq_ids = &seq;
    a.draft_ids = d_draft;
    a.mode = SJ_MODE_GREEDY;
    a.temperature = 1.f;
    a.theta_override = -1.f;
    a.commit = 1;
    const int before = kv->len_hi[seq];
    if (c >= 2) {
      // block [x_i, x_{i+1} .. x_{i+c-1}]: the c - 1 known continuations are the "drafts", all accepted
      a.gamma = c - 1;
      a.accept_all = 1;
      CU_TRY(cudaMemcpyAsync(d_draft, tokens + i + 1, sizeof(int) * (c - 1), cudaMemcpyHostToDevice, t->stream));
    } else {
      // a lone last token: a block of two rows whose second row (a dummy draft) is rejected outright
      a.gamma = 1;
      a.use_align = 0;
      a.use_judge = 0;
      CU_TRY(cudaMemsetAsync(d_draft, 0, sizeof(int), t->stream));
    }
    if ((st = sj_verify(t, kv, &a, &o)) != SJ_OK) return st;
    kv->len_hi[seq] = before + c;   // the host knows exactly how many rows such a block keeps
    kv->exact[seq] = 1;
    i += c;
  }
  if (next_token) {
    CU_TRY(cudaMemcpyAsync(next_token, o.next_token, sizeof(int), cudaMemcpyDeviceToHost, t->stream));
    CU_TRY(cudaStreamSynchronize(t->stream));
  }
  return SJ_OK;
}

// ---------------------------------------------------------------------------------------------
// standalone skinny GEMM
// ---------------------------------------------------------------------------------------------
__global__ void k_sum_slots(const float* __restrict__ P, SplitPlan sp, size_t slot_stride, int R, int N, float* __restrict__ Y) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)R * N) return;
  Y[i] = reduce_partials(P, sp, slot_stride, N, (int)(i / N), (int)(i % N));
}

extern "C" sj_status sj_gemm_skinny(int dtype, int impl, int R, int N, int K, const void* a, const void* w, float* y,
                                    void* cuda_stream) {
  if (!a || !w || !y) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (R <= 0 || R > SJ_MAX_ROWS || N <= 0 || K <= 0 || K % 8) return fail(SJ_ERR_SHAPE, "bad GEMM shape");
  cudaStream_t s = (cudaStream_t)cuda_stream;
  if (impl == 0) {
    GemmSegs g{{w, nullptr, nullptr}, {N, 0, 0}, 1};
    if (dtype == SJ_DTYPE_BF16)
      CU_TRY(launch(k_gemm_simt<bf16, 8>, dim3((N + 7) / 8), dim3(256), 0, s, false, (const bf16*)a, g, y, R, N, K, 1));
    else if (dtype == SJ_DTYPE_F32)
      CU_TRY(launch(k_gemm_simt<float, 8>, dim3((N + 7) / 8), dim3(256), 0, s, false, (const float*)a, g, y, R, N, K, 1));
    else
      return fail(SJ_ERR_INVALID_ARG, "unknown dtype");
    return SJ_OK;
  }
  if (impl != 1) return fail(SJ_ERR_INVALID_ARG, "unknown impl");
  if (dtype != SJ_DTYPE_BF16 || K % kBK) return fail(SJ_ERR_UNSUPPORTED, "tensor-core GEMM needs bf16 and K %% 64 == 0");
  cudaDeviceProp prop;
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  CU_TRY(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return fail(SJ_ERR_UNSUPPORTED, "built for sm_100a");
  sj_target tmp;  // borrowed only for its plumbing fields
  tmp.stream = s;
  tmp.sm_count = prop.multiProcessorCount;
  tmp.dm.V = N;
  memset(&tmp.work, 0, sizeof(tmp.work));
  TcSite site;
  int seg[1] = {N};
  sj_status st = setup_site(&tmp, site, 1, seg, K, false);
  auto cleanup = [&]() { for (void* p : tmp.owned) counted_free(p); };
  if (st != SJ_OK) { cleanup(); return st; }
  float* P = nullptr;
  int* status = nullptr;
  if ((st = dev_alloc(&tmp, &P, (size_t)site.max_slots * R * N)) != SJ_OK) { cleanup(); return st; }
  if ((st = dev_alloc(&tmp, &status, 1)) != SJ_OK) { cleanup(); return st; }
  cudaMemsetAsync(status, 0, sizeof(int), s);
  tmp.work.P = P;
  tmp.work.status = status;
  CUtensorMap mA, mW;
  RowGeom g = row_geom(R);
  if ((st = make_map(&mA, a, R, K, g.nblk)) != SJ_OK) { cleanup(); return st; }
  if ((st = make_map(&mW, w, N, K, kTileN)) != SJ_OK) { cleanup(); return st; }
  cudaError_t e = cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = launch_tc(&tmp, site, &mA, &mW, nullptr, nullptr, R, false, false);
  if (e == cudaSuccess)
    e = launch(k_sum_slots, dim3((unsigned)(((size_t)R * N + 255) / 256)), dim3(256), 0, s, false, (const float*)P,
               SplitPlan{site.d_tile_slots, site.n_tiles}, (size_t)R * N, R, N, y);
  int hstatus = 0;
  if (e == cudaSuccess) e = cudaMemcpyAsync(&hstatus, status, sizeof(int), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  cleanup();
  if (e != cudaSuccess) { cudaGetLastError(); return fail(SJ_ERR_CUDA, "sj_gemm_skinny: %s", cudaGetErrorString(e)); }
  if (hstatus != 0) return fail(SJ_ERR_TIMEOUT, "a bounded device-side wait ran out");
  return SJ_OK;
}

// ---------------------------------------------------------------------------------------------
// skinny GEMM that allocates nothing (see sj_gemm_skinny_noalloc in sj.h)
// ---------------------------------------------------------------------------------------------
// Scratch shared by every call on a device.  Layout: [0, 256) device status word; [256, slots_end)
// the per-tile slot table; from slots_end (256-byte aligned) the fp32 partial sums [slot][R][N].
// In host code `g_noalloc_scratch` is only a handle for cudaGetSymbolAddress(); the device address is
// looked up once per device and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SJ_NOALLOC_SCRATCH_BYTES];

constexpr int kNoAllocMaxDevices = 64;
static unsigned char* g_noalloc_ptr[kNoAllocMaxDevices] = {nullptr};
static int g_noalloc_sms[kNoAllocMaxDevices] = {0};
static std::mutex g_noalloc_mu;

// Same table as build_tile_slots(), computed on the device so that no host-to-device copy is needed.
__global__ void k_noalloc_tile_slots(int2* __restrict__ slots, int n_tiles, int KB, int G) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_tiles) return;
  const long long U = (long long)n_tiles * KB, t_lo = (long long)t * KB, t_hi = t_lo + KB;
  int first = -1, cnt = 0;
  for (int c = 0; c < G; ++c) {
    const long long lo = (long long)c * U / G, hi = (long long)(c + 1) * U / G;
    if (hi <= lo || lo >= t_hi || hi <= t_lo) continue;
    if (first < 0) first = c;
    cnt = c - first + 1;
  }
  slots[t] = make_int2(first, cnt);
}

extern "C" sj_status sj_gemm_skinny_noalloc(int R, int N, int K, const void* a, const void* w, float* y,
                                            void* cuda_stream) {
  if (!a || !w || !y) return fail(SJ_ERR_INVALID_ARG, "null argument");
  if (R <= 0 || R > SJ_MAX_ROWS || N <= 0 || K <= 0 || K % kBK) return fail(SJ_ERR_SHAPE, "bad GEMM shape (K must be a multiple of 64)");
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kNoAllocMaxDevices) return fail(SJ_ERR_UNSUPPORTED, "device ordinal %d not supported", dev);
  unsigned char* scratch = nullptr;
  int sms = 0;
  {
    // first call on this device (which is current): resolve the scratch array's device address
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
      int major = 0;
      CU_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
      if (major != 10) return fail(SJ_ERR_UNSUPPORTED, "built for sm_100a");
      CU_TRY(cudaDeviceGetAttribute(&g_noalloc_sms[dev], cudaDevAttrMultiProcessorCount, dev));
      void* p = nullptr;
      CU_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
      if (!p) return fail(SJ_ERR_CUDA, "cudaGetSymbolAddress returned a null scratch address");
      CU_TRY(cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
      g_noalloc_ptr[dev] = reinterpret_cast<unsigned char*>(p);
    }
    scratch = g_noalloc_ptr[dev];
    sms = g_noalloc_sms[dev];
  }
  // work split, as in sj_gemm_skinny()
  TcSite site;
  site.nseg = 1; site.K = K; site.KB = K / kBK; site.lm = false; site.N = N;
  site.n_tiles = (N + kTileN - 1) / kTileN;
  site.seg_tile_end[0] = site.seg_tile_end[1] = site.seg_tile_end[2] = site.n_tiles;
  site.G = (int)std::min<long long>((long long)site.n_tiles * site.KB, sms);
  {
    std::vector<int2> host_slots;  // host copy, only to learn the deepest split
    build_tile_slots(site.n_tiles, site.KB, site.G, host_slots, site.max_slots);
  }
  const size_t slots_end = 256 + (((size_t)site.n_tiles * sizeof(int2) + 255) & ~(size_t)255);
  const size_t need = slots_end + (size_t)site.max_slots * R * N * sizeof(float);
  if (need > (size_t)SJ_NOALLOC_SCRATCH_BYTES)
    return fail(SJ_ERR_SHAPE, "sj_gemm_skinny_noalloc: R=%d N=%d K=%d needs %zu bytes of scratch, the static array holds %zu",
                R, N, K, need, (size_t)SJ_NOALLOC_SCRATCH_BYTES);
  int* status = reinterpret_cast<int*>(scratch);
  site.d_tile_slots = reinterpret_cast<int2*>(scratch + 256);
  float* P = reinterpret_cast<float*>(scratch + slots_end);
  // the array keeps the previous call's contents: the status word must start at zero; the slot table and
  // every partial sum that is read are rewritten below before they are read
  CU_TRY(cudaMemsetAsync(status, 0, 256, s));
  CU_TRY(launch(k_noalloc_tile_slots, dim3((site.n_tiles + 127) / 128), dim3(128), 0, s, false, site.d_tile_slots,
                site.n_tiles, site.KB, site.G));
  sj_target tmp;  // borrowed for its plumbing fields only; owns nothing
  tmp.stream = s;
  tmp.sm_count = sms;
  tmp.dm.V = N;
  memset(&tmp.work, 0, sizeof(tmp.work));
  tmp.work.P = P;
  tmp.work.status = status;
  CUtensorMap mA, mW;
  RowGeom g = row_geom(R);
  sj_status st;
  if ((st = make_map(&mA, a, R, K, g.nblk)) != SJ_OK) return st;
  if ((st = make_map(&mW, w, N, K, kTileN)) != SJ_OK) return st;
  CU_TRY(launch_tc(&tmp, site, &mA, &mW, nullptr, nullptr, R, false, false));
  CU_TRY(launch(k_sum_slots, dim3((unsigned)(((size_t)R * N + 255) / 256)), dim3(256), 0, s, false, (const float*)P,
                SplitPlan{site.d_tile_slots, site.n_tiles}, (size_t)R * N, R, N, y));
  int hstatus = 0;
  CU_TRY(cudaMemcpyAsync(&hstatus, status, sizeof(int), cudaMemcpyDeviceToHost, s));
  CU_TRY(cudaStreamSynchronize(s));
  if (hstatus != 0) return fail(SJ_ERR_TIMEOUT, "a bounded device-side wait ran out");
  return SJ_OK;
}
