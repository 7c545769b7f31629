// The whole verification step as ONE persistent cooperative kernel (bf16 models, up to kMegaMaxRows
// block rows): one thread block per SM, every phase of every layer executed by the same blocks with a
// device-wide barrier between dependent phases.
//
// Why: at batch 1 the step is a chain of ~200 dependent phases of 10-100 us each, and the only thing
// that takes time is streaming 15 GB of weights (plus the KV cache) from HBM.  Weights and cached K/V
// do not depend on activations, so each block's producer warp streams ITS share of every phase's
// weights and cache tiles through one shared-memory ring without ever stopping at a phase boundary;
// consumers (the tcgen05 issuer, the attention warps) catch up after each barrier.  HBM stays busy
// across barriers for as long as the ring has free stages.
//
// Roles per block (384 threads):
//   warp 0      weight / cache-tile producer (TMA into the ring; never stops at a phase boundary)
//   warp 1      tcgen05.mma issuer, owns the TMEM allocation
//   warps 2, 3  activation producers: TMA of the activation K-slices (alternate units), gated by the device-wide barrier
//   warps 4..11 workers: all eight drain TMEM (fused epilogues, two groups of four warps) and run attention,
//               the combine, the embedding and the final acceptance phase
//
// GEMM phases: work units are (128-feature tile, 64-wide K block) in tile-major order, dealt evenly to
// the blocks (stream-K).  Partial sums of a tile that several blocks share travel as 64-bit words {fp32
// value, phase number} that the finishing block polls (no flag, no fence); the fused epilogues:
//   QKV   -> scale by 1/rms, bias, rotary embedding; queries (fp16, pre-scaled) to the query buffer, K and V
//            rows into the cache pages (bf16) and into the step's own fp16 side buffer
//   O     -> residual add, fp32 residual stream, next GEMM input planes (x * gain, hi/lo bf16), per-tile
//            sum of squares (the 1/rms factor is applied by the consumer's epilogue: it is a row scalar)
//   gate/up (tiles interleave 64 gate and 64 up features) -> silu(g) * u -> down-projection input planes
//   down  -> as O
//   LM head -> softmax statistics per (vocabulary tile, row), logit of the drafted token
// Attention: its cache tiles travel through the same ring.  Two implementations, chosen per launch: fp16 mma.sync in
// the worker warps (sj_attn_tc.cuh), or -- head dimension 128, at most 64 query rows per KV head and sequence --
// tcgen05 (the routines at the end of sj_attn_t5.cuh; ring stages of at least 32 KiB): warps 1 and 2 issue the MMAs of
// the even and the odd 128-key tiles, four worker warps run the softmax on tensor memory, the other four the causal tails; the queries sit in an area of their own
// after the ring, the accumulators alias the GEMM phases' tensor-memory columns.
//
// Every wait is bounded; the first one to run out raises a device-wide abort word that all other waits
// poll, so that a logic error ends the kernel with SJ_ERR_TIMEOUT instead of hanging the GPU.
#pragma once

#include "sj_attn_tc.cuh"
#include "sj_gemm_tc.cuh"
#include "sj_attn_t5.cuh"

namespace sj {

constexpr int kMegaThreads = 384;
constexpr int kMegaWorkers = 256;
constexpr int kMegaMaxLayers = 32;   // per launch (tensor maps travel as kernel parameters)
constexpr int kMegaMaxRows = 80;
constexpr int kMegaMaxStages = 12;
constexpr uint32_t kMegaSpin = 1u << 22;
constexpr int kMegaRegsLight = 80;    // registers per thread of warps 0..3 after reallocation
constexpr int kMegaRegsHeavy = 208;   // registers per thread of the worker warps
// The block is launched with 168 registers per thread (384 threads); the workers' increase can only be granted
// out of what the four light warps gave back, otherwise `setmaxnreg.inc` waits for ever.
static_assert(128 * kMegaRegsLight + 256 * kMegaRegsHeavy <= kMegaThreads * 168, "register reallocation exceeds the block's registers");
constexpr int kMegaTraceBarriers = 1024;
constexpr int kMegaTraceSites = 512;
constexpr int kMegaTraceAllBarriers = 32;   // barriers whose arrival / release time every block records
constexpr int kMegaTraceRelease = 2 * kMegaTraceBarriers + 16 * kMegaTraceSites;   // [barrier][256 blocks]
constexpr int kMegaTraceArrive = kMegaTraceRelease + kMegaTraceAllBarriers * 256;
constexpr int kMegaTraceEntries = kMegaTraceArrive + kMegaTraceAllBarriers * 256;

enum MegaSite { SITE_QKV = 0, SITE_O = 1, SITE_GU = 2, SITE_DOWN = 3, SITE_LM = 4 };

struct MegaMaps {
  CUtensorMap wq[kMegaMaxLayers], wk[kMegaMaxLayers], wv[kMegaMaxLayers], wo[kMegaMaxLayers];
  CUtensorMap wg[kMegaMaxLayers], wu[kMegaMaxLayers], wd[kMegaMaxLayers];   // wg, wu: boxes of 64 rows
  CUtensorMap lm, pool, a_d, a_q, a_f;
};

struct MegaLayerPtrs {
  const bf16 *bq, *bk, *bv;   // null without qkv_bias
  const bf16* gain_ffn;       // RMSNorm gain applied to the O projection's output (input of gate/up)
  const bf16* gain_next;      // gain applied to the down projection's output (next layer / final norm)
};

struct MegaParams {
  int l0, l1, do_embed, do_lm;
  int B, rows, R, Rp;
  int stages, stage_bytes;
  uint32_t tmem_cols;
  const MegaLayerPtrs* lp;    // [n_layers], device
  const bf16* embed;
  const bf16* lm_head;        // rows of the LM head (top-k test: the drafted tokens' logits are computed ahead of the head)
  const bf16* gain0;          // first layer's attention-norm gain
  float* sumsq;               // [2][d/128][kMegaMaxRows]
  // Split-K partial sums, [blocks][Rp][128] words of 64 bits: the fp32 value in the low half and, in the
  // high half, the number of the GEMM phase that wrote it (1, 2, ... within a launch).  A word is stored and
  // loaded as one 64-bit access, so a reader that sees the phase number it expects also sees the value:
  // no flag, no fence, and the reader polls the data itself.
  // Two slots per block ([block][2][Rp][128]): slot 1 for the tile whose first K block it holds, slot 0 otherwise.
  unsigned long long* pbuf;   //                               }
  unsigned* gbar;             // device-wide barrier counter   } zeroed before every launch
  int* abort_g;               // device-wide abort word        }
  int n_tail_base;
  int att_precise_layers;     // layers [0, n) run the attention with two-term (hi + lo fp16) queries and probabilities
  int q_area_bytes;           // tcgen05 attention: bytes of the query area between the ring and the control block
  // optional timeline (global-timer nanoseconds), block `trace_block`:
  //   [2k], [2k+1]                      arrival at / release from device-wide barrier k (k >= 1)
  //   [2*kMegaTraceBarriers + 8*s + e]  event e of GEMM phase s: 0 activation producer released, 1 its last
  //   load issued, 2 first stage ready at the MMA issuer, 3 last MMA committed, 4 last accumulator seen by the
  //   epilogue, 5 split-K partial sums gathered, 6 epilogue done, 7 weight producer issued the last load
  // and of every block: [kMegaTraceRelease + 256*k + block], [kMegaTraceArrive + 256*k + block] for k < 32
  unsigned long long* trace;
  unsigned trace_block;       // the block that writes the timeline
};

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
  return t;
}
// The timeline is compiled in only in the kernel's tracing instantiation (`kTr` in scope): the timer reads
// are volatile and hold back the compiler's scheduling even when no trace is taken (1.7 % of a step).
#define MEGA_EV(sidx, k)                                                                             \
  do {                                                                                               \
    if constexpr (kTr)                                                                               \
    if (p.trace && blockIdx.x == p.trace_block && (sidx) < kMegaTraceSites)                                      \
      p.trace[2 * kMegaTraceBarriers + (sidx) * 8 + (k)] = global_timer_ns();                        \
  } while (0)

// second event set (fine-grained epilogue timing): block 1 records its contributor-side events, block 0 its
// owner-side ones, at [2*kMegaTraceBarriers + 8*kMegaTraceSites + 8*s + e]
#define MEGA_EV2(blk, sidx, k)                                                                       \
  do {                                                                                               \
    if constexpr (kTr)                                                                               \
    if (p.trace && blockIdx.x == p.trace_block + (blk) && (sidx) < kMegaTraceSites)                                  \
      p.trace[2 * kMegaTraceBarriers + 8 * kMegaTraceSites + (sidx) * 8 + (k)] = global_timer_ns();  \
  } while (0)

struct MegaCtl {
  uint64_t full[kMegaMaxStages], empty[kMegaMaxStages], tmem_full[2], tmem_empty[2];
  int cons_cnt[kMegaMaxStages];
  uint32_t tmem_base;
  int abort_flag;
  int bars_passed;
  A5Bars a5;                   // tcgen05 attention: score / probability / output hand-offs
  uint64_t a5_pair[2];         // ... and the barrier of each lane quarter's two softmax warps
  int bcast[6];   // [2 * group + accumulator]: the group's wait on that accumulator succeeded; [4], [5] spare
  float inv[kMegaMaxRows];
  float zd[kMegaMaxRows];      // top-k test: raw logit of each row's drafted token, computed before the LM head
  int row_b[kMegaMaxRows], row_j[kMegaMaxRows], row_page[kMegaMaxRows], row_slot[kMegaMaxRows], tgt_tok[kMegaMaxRows];
  int row_qoff[kMegaMaxRows];         // element offset of row r's queries in the query buffer, without the head part
  int row_nkvoff[kMegaMaxRows];       // element offset of row r in the fp16 copy of the step's own K/V rows, without head / K|V part
  long long row_kvoff[kMegaMaxRows];  // element offset of row r's slot in its cache page, without layer / K|V / head part
  float red[2][4][8];          // [group][warp][row of the chunk]
  RowStat wstat[2][4][8];
  RowStat rs[kMaxGamma + 1];
  float score[kMaxGamma + 1];
  AttPlan plan;
  int att_pages[kAttPageCache];   // page ids of this block's first ring tiles (the same in every layer)
  union {
    float exch[2][128][9];      // [group][feature][row of the chunk]
    float a5_mx[2][2][64];      // tcgen05 attention: [tile parity][key half][query row] maxima / sums of a row's two threads
    RowStat sred[kMegaWorkers];
  } u;
};

// The tcgen05 attention's M = 128 descriptors read up to 16 KiB past the last half of the query area, which this
// block follows: those bytes must be the kernel's own.
static_assert(sizeof(MegaCtl) >= 16384, "the control block no longer covers the query area's over-read");

struct SiteInfo {
  int n_tiles, KB;
};
__host__ __device__ __forceinline__ SiteInfo site_info(int site, const Dims& dm, int c, int G) {
  SiteInfo s;
  const int qd = dm.Hq * dm.hd, kd = dm.Hkv * dm.hd;
  switch (site) {
    case SITE_QKV: s.n_tiles = (qd + 2 * kd) / kTileN; s.KB = dm.d / kBK; break;
    case SITE_O: s.n_tiles = dm.d / kTileN; s.KB = qd / kBK; break;
    case SITE_GU: s.n_tiles = dm.F / 64; s.KB = dm.d / kBK; break;
    case SITE_DOWN: s.n_tiles = dm.d / kTileN; s.KB = dm.F / kBK; break;
    default: s.n_tiles = (dm.V + kTileN - 1) / kTileN; s.KB = dm.d / kBK; break;
  }
  return s;
}
// Block that owns unit u of a stream-K site.
__device__ __forceinline__ int unit_owner(unsigned u, unsigned U, int G) {
  unsigned c = u * (unsigned)G / U;
  while ((c + 1) * U / (unsigned)G <= u) ++c;
  return (int)c;
}
// Whether block c owns at least one unit when U units are dealt to G blocks.
__device__ __forceinline__ bool has_units(int c, unsigned U, int G) {
  return (unsigned)(c + 1) * U / (unsigned)G > (unsigned)c * U / (unsigned)G;
}

// How a site's units are dealt.  A "group" is CS consecutive blocks that share segments (CS = 1 everywhere
// at present: a B200 holds only 33 clusters of four of these blocks, and streaming with 132 of its 148 SMs
// cost more than an exchange through distributed shared memory saved).  Groups take [g*U/n, (g+1)*U/n);
// every maximal run of units of one tile inside a group's range is a segment, and block `rank` of the group
// takes the K blocks [kb0 + rank*len/CS, kb0 + (rank+1)*len/CS) of it.
// Unit counts stay far below 2^24 (at most a few hundred tiles of a few hundred K blocks), so all of this
// is 32-bit arithmetic: 64-bit division is a long inlined routine and these helpers sit in every role.
struct SiteSplit {
  int n_tiles, KB, CS, rank, grp, ngrp;
  unsigned U, g_lo, g_hi;
};
__device__ __forceinline__ SiteSplit site_split(int site, const Dims& dm, int c, int G) {
  SiteSplit s;
  const SiteInfo t = site_info(site, dm, 0, 1);
  s.n_tiles = t.n_tiles;
  s.KB = t.KB;
  s.CS = 1;
  s.ngrp = G / s.CS;
  s.grp = c / s.CS;
  s.rank = c % s.CS;
  s.U = (unsigned)s.n_tiles * (unsigned)s.KB;
  // every site is dealt by units, the LM head too: whole vocabulary tiles would leave a quarter of the
  // blocks one tile short (1002 tiles on 148 blocks) and idle for 15 % of the phase
  s.g_lo = (unsigned)s.grp * s.U / (unsigned)s.ngrp;
  s.g_hi = (unsigned)(s.grp + 1) * s.U / (unsigned)s.ngrp;
  return s;
}
struct Seg { int tile, kb0, len, a, b; };
__device__ __forceinline__ bool seg_next(const SiteSplit& s, unsigned& u, Seg& g) {
  if (u >= s.g_hi) return false;
  g.tile = (int)(u / (unsigned)s.KB);
  g.kb0 = (int)(u % (unsigned)s.KB);
  g.len = (int)min((unsigned)(s.KB - g.kb0), s.g_hi - u);
  g.a = g.kb0 + s.rank * g.len / s.CS;
  g.b = g.kb0 + (s.rank + 1) * g.len / s.CS;
  u += g.len;
  return true;
}
__device__ __forceinline__ int site_units(const SiteSplit& s) {
  unsigned u = s.g_lo;
  Seg g;
  int n = 0;
  while (seg_next(s, u, g)) n += g.b - g.a;
  return n;
}

// The step as a list of phases: per layer QKV, attention (+ combine, which streams nothing), O, gate/up,
// down; then the LM head.  One call site per callback: the callbacks are large and get inlined, and the
// kernel has to fit the instruction cache.
__device__ __forceinline__ int mega_n_phases(const MegaParams& p) { return 5 * (p.l1 - p.l0) + (p.do_lm ? 1 : 0); }
// phase index -> (site or -1 for attention, layer)
__device__ __forceinline__ void mega_phase(const MegaParams& p, int ph, int& site, int& l) {
  const int nl = p.l1 - p.l0;
  if (ph >= 5 * nl) { site = SITE_LM; l = p.l1 - 1; return; }
  l = p.l0 + ph / 5;
  const int k = ph % 5;
  site = k == 0 ? SITE_QKV : k == 1 ? -1 : k == 2 ? SITE_O : k == 3 ? SITE_GU : SITE_DOWN;
}
// Position in the ring: stage index and how many times the ring has wrapped, advanced without divisions.
struct RingPos {
  int s, r, NS;
  __device__ __forceinline__ void advance(int n) {   // n may exceed NS (skipping a phase's stages)
    s += n;
    if (s >= NS) { r += s / NS; s %= NS; }
  }
  __device__ __forceinline__ void next() {
    if (++s == NS) { s = 0; ++r; }
  }
};
template <typename FSite, typename FAtt>
__device__ __forceinline__ void mega_walk(const MegaParams& p, FSite fsite, FAtt fatt) {
  const int n = mega_n_phases(p);
  for (int ph = 0; ph < n; ++ph) {
    int site, l;
    mega_phase(p, ph, site, l);
    if (site < 0) fatt(l);
    else fsite(site, l);
  }
}

__device__ __forceinline__ void bar_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ unsigned ld_relaxed_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_relaxed_add(unsigned* p, unsigned v) {
  asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

// Bounded wait on a shared-memory barrier that also watches the device-wide abort word.
__device__ __forceinline__ bool mega_wait(uint32_t bar, uint32_t parity, MegaCtl* ctl, const MegaParams& p, int* status,
                                          int where, int extra) {
  return att_mbar_wait(bar, parity, &ctl->abort_flag, status, p.abort_g, where, extra);
}
// Bounded spin (relaxed polls; the caller fences after success) until *word (device memory, written by
// other blocks) reaches `target`.
__device__ __forceinline__ bool mega_spin_ge(const unsigned* word, unsigned target, MegaCtl* ctl, const MegaParams& p,
                                             int* status, int where, int extra, uint32_t limit = kMegaSpin) {
  volatile int* af = &ctl->abort_flag;
  volatile int* ag = p.abort_g;
  for (uint32_t i = 0; i < limit; ++i) {
    if (ld_relaxed_u32(word) >= target) return true;
    if (i > 16) {
      if (*af) return false;
      if ((i & 63) == 0 && *ag) { *af = 1; return false; }
      if (i > 4096) __nanosleep(64);
    }
  }
  *af = 1;
  att_note_timeout(ag, where, extra);
  *ag = 1;
  atomicCAS(status, DEV_OK, DEV_TIMEOUT);
  return false;
}

// Device-wide barrier for the 256 workers of every block.  Returns false once the step is aborting.
// Block-level barrier, then one thread publishes (fence, arrive) and waits (poll, fence): the fences are
// cumulative over what the block barrier ordered before them.
template <bool kTr>
__device__ __forceinline__ bool mega_grid_sync(MegaCtl* ctl, const MegaParams& p, int* status, int& nbar, int wt) {
  fence_proxy_async();   // this phase's generic-proxy stores are read by other blocks' TMA loads
  bar_sync(1, kMegaWorkers);
  ++nbar;
  if (wt == 0) {
    const bool tr = kTr && p.trace && blockIdx.x == p.trace_block && nbar < kMegaTraceBarriers;
    if (tr) p.trace[2 * nbar] = global_timer_ns();
    if (kTr && p.trace && nbar < kMegaTraceAllBarriers) p.trace[kMegaTraceArrive + nbar * 256 + blockIdx.x] = global_timer_ns();
    if (!ctl->abort_flag) {
      __threadfence();
      red_relaxed_add(p.gbar, 1u);
      mega_spin_ge(p.gbar, (unsigned)nbar * gridDim.x, ctl, p, status, 8, nbar);
    }
    __threadfence();
    if (tr) p.trace[2 * nbar + 1] = global_timer_ns();
    if (kTr && p.trace && nbar < kMegaTraceAllBarriers) p.trace[kMegaTraceRelease + nbar * 256 + blockIdx.x] = global_timer_ns();
    *reinterpret_cast<volatile int*>(&ctl->bars_passed) = nbar;
  }
  bar_sync(1, kMegaWorkers);
  return *reinterpret_cast<volatile int*>(&ctl->abort_flag) == 0;
}

// Bounded wait (shared-memory polling) until the block's workers have passed `need` device-wide barriers.
__device__ __forceinline__ bool mega_wait_bars(int need, MegaCtl* ctl, const MegaParams& p, int* status, int where) {
  volatile int* bp = &ctl->bars_passed;
  volatile int* af = &ctl->abort_flag;
  for (uint32_t i = 0; i < kMegaSpin; ++i) {
    if (*bp >= need) return true;
    if (*af) return false;
    if (i > 64) __nanosleep(32);
  }
  ctl->abort_flag = 1;
  att_note_timeout(p.abort_g, where, need);
  *p.abort_g = 1;
  atomicCAS(status, DEV_OK, DEV_TIMEOUT);
  return false;
}

// TMA loads of one weight unit into a ring stage.
__device__ __forceinline__ void mega_issue_w(const MegaMaps& mp, int site, int li, const Dims& dm, int tile, int kb,
                                             uint32_t dst, uint32_t bar, uint64_t pol) {
  switch (site) {
    case SITE_QKV: {
      const int tq = dm.Hq * dm.hd / kTileN, tk = dm.Hkv * dm.hd / kTileN;
      if (tile < tq) tma_load_2d(dst, &mp.wq[li], bar, kb * kBK, tile * kTileN, pol);
      else if (tile < tq + tk) tma_load_2d(dst, &mp.wk[li], bar, kb * kBK, (tile - tq) * kTileN, pol);
      else tma_load_2d(dst, &mp.wv[li], bar, kb * kBK, (tile - tq - tk) * kTileN, pol);
      break;
    }
    case SITE_O: tma_load_2d(dst, &mp.wo[li], bar, kb * kBK, tile * kTileN, pol); break;
    case SITE_GU:
      tma_load_2d(dst, &mp.wg[li], bar, kb * kBK, tile * 64, pol);
      tma_load_2d(dst + 8192u, &mp.wu[li], bar, kb * kBK, tile * 64, pol);
      break;
    case SITE_DOWN: tma_load_2d(dst, &mp.wd[li], bar, kb * kBK, tile * kTileN, pol); break;
    default: tma_load_2d(dst, &mp.lm, bar, kb * kBK, tile * kTileN, pol); break;
  }
}

// ---------------------------------------------------------------------------------------------
// fused epilogues.  All eight worker warps take part, as two groups of four warps (a warp reads the
// accumulator lanes 32 * (warp % 4) .. + 31, so either group covers the tile's 128 features): of every 16
// block rows group 0 takes the first half of those that exist and group 1 the rest (5 + 4 at 9 rows).  One warp per scheduler runs a long dependent instruction chain at a fraction of an instruction
// per cycle, so halving the rows per thread nearly halves the time between the last MMA and the barrier.
// Each group has its own named barrier (2 + group, 128 threads) and its own exchange buffers.
// ---------------------------------------------------------------------------------------------
// Which of the two epilogue groups handles block row r: the rows of every 16-row chunk are halved.
__device__ __forceinline__ int mega_row_group(int r, int R) {
  const int c16 = r & ~15, n16 = min(16, R - c16);
  return (r - c16) >= ((n16 + 1) >> 1) ? 1 : 0;
}

// NS: row slots a thread unrolls per chunk (4, 6 or 8): at least the rows a group gets of a 16-row chunk.
// Every slot's instructions issue whether its row exists or not, so the kernel is instantiated for the
// slot counts 4 (up to 8 block rows), 6 (up to 12) and 8.
template <int HD, int NS, bool kTr>
__device__ __forceinline__ void mega_epilogue(int site, int l, int gseq, int& seg, MegaCtl* ctl, const MegaParams& p, const StepArgs* __restrict__ args, const KvView& kv,
                                              const Work& w, const Dims& dm, int wt) {
  const int et = wt & 127, grp = wt >> 7, bar_id = 2 + grp;
  const int sidx = gseq - 1;
  const int R = p.R, Rp = p.Rp, rows = p.rows;
  const int quarter = et >> 5, lane = et & 31;
  const SiteSplit ss = site_split(site, dm, blockIdx.x, gridDim.x);
  if (ss.g_hi <= ss.g_lo) return;   // nothing to do in this phase
  const int c = ss.grp, G = ss.ngrp;   // split-K partners across groups are addressed by group
  const unsigned U = ss.U;
  const int nt128 = dm.d / kTileN;
  const MegaLayerPtrs lp = p.lp[l];
  // 1/rms of this phase's input rows (the planes hold x * gain; the scalar is applied here).  One warp
  // per row, lanes over the column tiles, fixed shuffle tree: all loads of a row are in flight together.
  if (site == SITE_QKV || site == SITE_GU || site == SITE_LM) {
    const int buf = (site == SITE_GU) ? 1 : 0;
    for (int r0 = quarter; r0 < R; r0 += 16) {
      float part[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int r = r0 + 4 * k;
        part[k] = 0.f;
        if (r < R && mega_row_group(r, R) == grp)
          for (int t = lane; t < nt128; t += 32) part[k] += __ldcg(p.sumsq + ((size_t)buf * nt128 + t) * kMegaMaxRows + r);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int r = r0 + 4 * k;
        const float s = warp_sum(part[k]);
        if (lane == 0 && r < R && mega_row_group(r, R) == grp) ctl->inv[r] = 1.0f / sqrtf(s / (float)dm.d + dm.eps);
      }
    }
    bar_sync(bar_id, 128);
  }
  const bool topk = site == SITE_LM && args->top_k >= 2;   // block-uniform
  if (topk) {
    // The LM head stores no logits, so the rank of a drafted token is counted tile by tile against its own
    // logit, which therefore has to exist first: one dot product per row (this group's rows, a warp each).
    const int gamma = rows - 1;
    for (int r = quarter; r < R; r += 4) {
      if (mega_row_group(r, R) != grp) continue;
      const int tok = ctl->tgt_tok[r];
      float z = 0.f;
      if (tok >= 0) z = planes_dot(reinterpret_cast<const bf16*>(w.A), R, dm.d, r, p.lm_head + (size_t)min(tok, dm.V - 1) * dm.d, lane) * ctl->inv[r];
      if (lane == 0) ctl->zd[r] = z;
    }
    (void)gamma;
    bar_sync(bar_id, 128);
  }
  const int qd = dm.Hq * dm.hd, kd = dm.Hkv * dm.hd, tq = qd / kTileN, tk = kd / kTileN;
  const float invT = (site == SITE_LM) ? args->inv_temperature : 1.f;
  float* dbg_logits = (site == SITE_LM) ? args->dbg_logits : nullptr;
  const float qscale = 1.4426950408889634f / sqrtf((float)HD);
  const int fl = et;   // feature inside the tile == TMEM lane

  int n_rs = 0, rs_tile0 = 0, rs_first0 = 0, rs_last0 = 0, rs_tile1 = 0, rs_first1 = 0, rs_last1 = 0;
  float rs_gn0 = 1.f, rs_gn1 = 1.f;
  unsigned u = ss.g_lo;
  Seg sg;
  while (seg_next(ss, u, sg)) {
    const int tile = sg.tile, kb0 = sg.kb0;
    const bool mine = sg.b > sg.a;   // this block computed a share of the segment
    const int acc = seg & 1, use = seg >> 1;
    const uint32_t taddr = ctl->tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 2 * Rp);

    // per-tile constants of the fused epilogues; their global loads are issued before any wait
    int kind = 0, head = 0, dim = 0;
    float bias = 0.f, gn = 1.f;
    if (site == SITE_QKV) {
      int fs;
      if (tile < tq) { kind = 0; fs = tile * kTileN + fl; }
      else if (tile < tq + tk) { kind = 1; fs = (tile - tq) * kTileN + fl; }
      else { kind = 2; fs = (tile - tq - tk) * kTileN + fl; }
      head = fs / HD;
      dim = fs % HD;
      const bf16* bp = kind == 0 ? lp.bq : (kind == 1 ? lp.bk : lp.bv);
      if (bp) bias = __bfloat162float(bp[fs]);
    } else if (site == SITE_O) {
      gn = __bfloat162float(lp.gain_ffn[tile * kTileN + fl]);
    } else if (site == SITE_DOWN) {
      gn = __bfloat162float(lp.gain_next[tile * kTileN + fl]);
    }

    const bool complete = (kb0 == 0) && (sg.len == ss.KB);
    // The O and down projections split a shared tile's epilogue by ROWS: the n blocks that hold K ranges of
    // the tile each finish R / n of its rows (all 128 features of them) and publish their sums of the other
    // rows, instead of one block finishing the whole tile while the others idle at the barrier.  (Needs every
    // block to hold units, so that the sharing blocks are consecutive.)
    const bool rowsplit = (site == SITE_O || site == SITE_DOWN) && !complete && U >= (unsigned)G;
    const bool owner = (kb0 == 0) && !rowsplit;
    int c_first = c, c_last = c;   // first and last of the blocks that share this tile
    if ((owner && !complete) || rowsplit) c_last = unit_owner((unsigned)(tile + 1) * (unsigned)ss.KB - 1u, U, G);
    if (rowsplit) c_first = unit_owner((unsigned)tile * (unsigned)ss.KB, U, G);
    if (et == 0) {
      int ok = 1;
      if (mine) ok = mega_wait(smem_u32(&ctl->tmem_full[acc]), use & 1, ctl, p, w.status, 6, gseq) ? 1 : 0;
      ctl->bcast[2 * grp + (seg & 1)] = ok;
    }
    bar_sync(bar_id, 128);
    if (!ctl->bcast[2 * grp + (seg & 1)]) return;
    tc_fence_after();
    if (et == 0) MEGA_EV(sidx, 4);

    for (int c16 = 0; c16 < Rp; c16 += 16) {
      // this group's rows of the 16-row chunk: the first or the second half of the rows that exist
      const int n16 = max(min(16, R - c16), 0), h16 = (n16 + 1) >> 1;
      const int c0 = c16 + (grp ? h16 : 0), nr = grp ? n16 - h16 : h16, rend = c0 + nr;
      float v[NS], xs[NS];
      float2 cs[NS];
      // every global load of this chunk is issued before anything waits on one of them
      if (owner && (site == SITE_O || site == SITE_DOWN)) {   // residual rows
        const int f = tile * kTileN + fl;
#pragma unroll
        for (int i = 0; i < NS; ++i) xs[i] = __ldcg(w.X + (size_t)max(min(c0 + i, rend - 1), 0) * dm.d + f);   // unpredicated: rows past R repeat the last row
      }
      if (owner && site == SITE_QKV && kind < 2) {            // rotary table rows
        const int ii = dim & (HD / 2 - 1);
#pragma unroll
        for (int i = 0; i < NS; ++i)
          cs[i] = __ldcg(w.rope + (size_t)max(min(c0 + i, rend - 1), 0) * (HD / 2) + ii);
      }
      if (mine) {
        float hi8[8], lo8[8];
        tc_ld8(taddr + c0, hi8);
        tc_ld8(taddr + Rp + c0, lo8);
#pragma unroll
        for (int i = 0; i < NS; ++i) v[i] = hi8[i] + lo8[i];
      } else {
#pragma unroll
        for (int i = 0; i < NS; ++i) v[i] = 0.f;
      }
      const unsigned long long tag = (unsigned long long)(unsigned)gseq << 32;
      if (et == 0 && owner) MEGA_EV2(0, sidx, 0);
      if (rowsplit) {   // publish every row; the rows are finished after the loop over the segments
        unsigned long long* dst = p.pbuf + ((size_t)(2 * c + (c == c_first ? 1 : 0)) * Rp + c0) * kTileN + fl;
#pragma unroll
        for (int i = 0; i < NS; ++i)
          if (i < nr) st_relaxed_u64(dst + (size_t)i * kTileN, tag | __float_as_uint(v[i]));
        continue;
      }
      if (!owner) {   // publish the partial sums, each with this phase's number
        unsigned long long* dst = p.pbuf + ((size_t)(2 * c) * Rp + c0) * kTileN + fl;
#pragma unroll
        for (int i = 0; i < NS; ++i)
          if (i < nr) st_relaxed_u64(dst + (size_t)i * kTileN, tag | __float_as_uint(v[i]));
        continue;
      }
      // The other blocks' shares of this tile: two blocks' words in flight at a time, all of them reloaded
      // until every one carries this phase's number, then added in group order (so the sum does not depend
      // on arrival order).  Often they were published long ago: a group's share of somebody else's tile is
      // the first thing it computes.  A wait that runs out raises the abort word and goes on with whatever
      // it read (the block leaves together at its next block-wide check).
      for (int cb = c + 1; cb <= c_last; cb += 2) {
        unsigned long long pw[2][NS];
        const unsigned long long* src[2];
        bool live[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int c2 = cb + k;
          live[k] = c2 <= c_last && has_units(c2, U, G);   // groups without units add nothing
          src[k] = p.pbuf + ((size_t)(2 * (live[k] ? c2 : c)) * Rp + c0) * kTileN + fl;
        }
        volatile int* af = &ctl->abort_flag;
        for (uint32_t spin = 0;; ++spin) {
          bool ok = true;
          // every load is issued before any result is looked at: rows past R read row 0 again (in
          // bounds, ignored below) instead of being predicated off, which would put a select after each load
#pragma unroll
          for (int k = 0; k < 2; ++k)
#pragma unroll
            for (int i = 0; i < NS; ++i) pw[k][i] = ld_relaxed_u64(src[k] + (size_t)(i < nr ? i : 0) * kTileN);
#pragma unroll
          for (int k = 0; k < 2; ++k)
#pragma unroll
            for (int i = 0; i < NS; ++i) ok = ok && (!live[k] || i >= nr || (pw[k][i] >> 32) == (tag >> 32));
          if (ok) break;
          if (spin > 16) {
            if (*af) break;
            if ((spin & 63) == 0 && *reinterpret_cast<volatile int*>(p.abort_g)) { *af = 1; break; }
            if (spin > 4096) __nanosleep(64);
            if (spin >= kMegaSpin) {
              *af = 1;
              att_note_timeout(p.abort_g, 7, gseq);
              *reinterpret_cast<volatile int*>(p.abort_g) = 1;
              atomicCAS(w.status, DEV_OK, DEV_TIMEOUT);
              break;
            }
          }
        }
#pragma unroll
        for (int k = 0; k < 2; ++k)
#pragma unroll
          for (int i = 0; i < NS; ++i) v[i] += (live[k] && i < nr) ? __uint_as_float((unsigned)pw[k][i]) : 0.f;
      }
      if (et == 0) MEGA_EV(sidx, 5);
      if (et == 0) MEGA_EV2(0, sidx, 1);
      if (site == SITE_QKV) {
        const int half = HD / 2;
#pragma unroll
        for (int i = 0; i < NS; ++i) {
          const int r = c0 + i;
          v[i] = v[i] * (r < rend ? ctl->inv[r] : 0.f) + bias;
        }
        if (kind < 2) {
#pragma unroll
          for (int i = 0; i < NS; ++i) ctl->u.exch[grp][fl][i] = v[i];
          bar_sync(bar_id, 128);
          const bool first = dim < half;
#pragma unroll
          for (int i = 0; i < NS; ++i) {
            const float xp = ctl->u.exch[grp][fl ^ half][i];
            v[i] = first ? v[i] * cs[i].x - xp * cs[i].y : v[i] * cs[i].x + xp * cs[i].y;
          }
          bar_sync(bar_id, 128);
        }
        if (et == 0) MEGA_EV2(0, sidx, 6);
        // query row (b, kvh, g, j) sits at ((b*Hq + head)*rows + j)*HD; a cache row at
        // ((((layer*n_pages + page)*2 + K|V)*Hkv + head)*page_size + slot)*HD: the per-row parts are tabulated
        if (kind == 0) {
          __half* qb = w.Qb + (size_t)head * rows * HD + dim;
          __half* ql = w.Qlo + (size_t)head * rows * HD + dim;
          const bool two_term = l < p.att_precise_layers;   // block-uniform
#pragma unroll
          for (int i = 0; i < NS; ++i)
            if (i < nr) {
              const float qv = v[i] * qscale;
              const __half hq = __float2half_rn(qv);
              qb[ctl->row_qoff[c0 + i]] = hq;
              if (two_term) ql[ctl->row_qoff[c0 + i]] = __float2half_rn(qv - __half2float(hq));
            }
        } else {
          bf16* kvb = reinterpret_cast<bf16*>(kv.pool) +
                      ((size_t)l * kv.n_pages * 2 * dm.Hkv + (size_t)(kind - 1) * dm.Hkv + head) * kv.page_size * HD + dim;
#pragma unroll
          for (int i = 0; i < NS; ++i)
            if (i < nr) kvb[ctl->row_kvoff[c0 + i]] = __float2bfloat16_rn(v[i]);
          __half* kn = w.KVn + (size_t)(head * 2 + kind - 1) * rows * HD + dim;
#pragma unroll
          for (int i = 0; i < NS; ++i)
            if (i < nr) kn[ctl->row_nkvoff[c0 + i]] = __float2half_rn(v[i]);
        }
      } else if (site == SITE_O || site == SITE_DOWN) {
        const int f = tile * kTileN + fl;
        const int buf = (site == SITE_O) ? 1 : 0;
        float ss[NS];
#pragma unroll
        for (int i = 0; i < NS; ++i) {
          const int r = c0 + i;
          ss[i] = 0.f;
          if (r < rend) {
            const float x = xs[i] + v[i];
            w.X[(size_t)r * dm.d + f] = x;
            store_act<bf16>(w.A, R, dm.d, r, f, x * gn);
            ss[i] = x * x;
          }
        }
        if (et == 0) MEGA_EV2(0, sidx, 2);
#pragma unroll
        for (int i = 0; i < NS; ++i)
          if (i < nr) ss[i] = warp_sum(ss[i]);   // block-uniform
        if (lane == 0) {
#pragma unroll
          for (int i = 0; i < NS; ++i) ctl->red[grp][quarter][i] = ss[i];
        }
        bar_sync(bar_id, 128);
        if (et < nr)
          p.sumsq[((size_t)buf * nt128 + tile) * kMegaMaxRows + c0 + et] =
              ctl->red[grp][0][et] + ctl->red[grp][1][et] + ctl->red[grp][2][et] + ctl->red[grp][3][et];
        bar_sync(bar_id, 128);
        if (et == 0) MEGA_EV2(0, sidx, 3);
      } else if (site == SITE_GU) {
#pragma unroll
        for (int i = 0; i < NS; ++i) {
          const int r = c0 + i;
          v[i] *= (r < rend ? ctl->inv[r] : 0.f);
        }
        if (fl >= 64) {
#pragma unroll
          for (int i = 0; i < NS; ++i) ctl->u.exch[grp][fl - 64][i] = v[i];
        }
        bar_sync(bar_id, 128);
        if (fl < 64) {
          const int f = tile * 64 + fl;
#pragma unroll
          for (int i = 0; i < NS; ++i) {
            const int r = c0 + i;
            if (r < rend) {
              const float g = v[i], up = ctl->u.exch[grp][fl][i];
              store_act<bf16>(w.H, R, dm.F, r, f, g / (1.0f + expf(-g)) * up);
            }
          }
        }
        bar_sync(bar_id, 128);
      } else {   // LM head
        const int n = tile * kTileN + fl;
#pragma unroll
        for (int i = 0; i < NS; ++i) {
          const int r = c0 + i;
          float z = -INFINITY;
          if (r < rend && n < dm.V) {
            const float raw = v[i] * ctl->inv[r];
            if (w.logits) w.logits[(size_t)r * dm.V + n] = raw;
            if (dbg_logits) dbg_logits[(size_t)r * dm.V + n] = raw;
            z = raw * invT;
            if (n == ctl->tgt_tok[r]) w.tgt_logit[r] = z;
          }
          float m = z;
          int arg = n;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, m, o);
            const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
            if (om > m || (om == m && oa < arg)) { m = om; arg = oa; }
          }
          float e = (z == -INFINITY) ? 0.f : expf(z - m);
          e = warp_sum(e);
          int before = 0;
          if (topk) {
            const int rr = min(r, R - 1), tg = ctl->tgt_tok[rr];
            const float raw = v[i] * ctl->inv[rr], zd = ctl->zd[rr];
            const bool bf = r < rend && n < dm.V && tg >= 0 && n != tg && (raw > zd || (raw == zd && n < tg));
            before = __popc(__ballot_sync(0xffffffffu, bf));
          }
          if (lane == 0) {
            RowStat st; st.m = m; st.s = e; st.arg = arg; st.pad = before;
            ctl->wstat[grp][quarter][i] = st;
          }
        }
        bar_sync(bar_id, 128);
        if (et < nr) {
          RowStat a = ctl->wstat[grp][0][et];
          a = stat_merge(a, ctl->wstat[grp][1][et]);
          a = stat_merge(a, ctl->wstat[grp][2][et]);
          a = stat_merge(a, ctl->wstat[grp][3][et]);
          w.stats[(size_t)tile * R + c0 + et] = a;
        }
        bar_sync(bar_id, 128);
      }
    }
    if (et == 0) MEGA_EV2(0, sidx, 7);
    if (mine) {
      tc_fence_before();
      mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
      ++seg;
    }
    if (rowsplit) {   // at most two per phase: the block's first and last segment
      if (n_rs == 0) { rs_tile0 = tile; rs_first0 = c_first; rs_last0 = c_last; rs_gn0 = gn; }
      else { rs_tile1 = tile; rs_first1 = c_first; rs_last1 = c_last; rs_gn1 = gn; }
      ++n_rs;
    }
  }
  // Row-split tiles (O and down projections): this block's rows of each shared tile.  Every sharing block
  // has published all its rows by now or will without waiting for anybody (publishing comes first in every
  // block), so the waits below cannot form a chain.  A row's sums are added in block order.
#pragma unroll 1
  for (int q = 0; q < n_rs; ++q) {
    const int tile = q ? rs_tile1 : rs_tile0, c_first = q ? rs_first1 : rs_first0, c_last = q ? rs_last1 : rs_last0;
    const float gn = q ? rs_gn1 : rs_gn0;
    const int n = c_last - c_first + 1, j = c - c_first;
    const int f = tile * kTileN + fl;
    const int buf = (site == SITE_O) ? 1 : 0;
    const unsigned long long tag = (unsigned long long)(unsigned)gseq << 32;
    volatile int* af = &ctl->abort_flag;
#pragma unroll 1
    for (int c16 = 0; c16 < Rp; c16 += 16) {
      const int n16 = max(min(16, R - c16), 0), h16 = (n16 + 1) >> 1;
      const int c0 = c16 + (grp ? h16 : 0), nr = grp ? n16 - h16 : h16;
      // Rows are dealt with weight 1 to the first and the last sharing block and weight 2 to the others:
      // the first block of one tile is as a rule the last block of the tile before, and finishes rows of both.
      const int wsum = 2 * n - 2, w_lo = j == 0 ? 0 : 2 * j - 1, w_hi = j == n - 1 ? wsum : 2 * j + 1;
      const int a = max(w_lo * R / wsum - c0, 0), b = min(w_hi * R / wsum - c0, nr);   // this block's rows of the chunk: [a, b)
#pragma unroll 1
      for (int i = a; i < b; i += 2) {   // two rows at a time: their loads share one round trip
        const int i1 = min(i + 1, b - 1);   // == i when the second row is absent: it repeats the first
        const int r0 = c0 + i, r1 = c0 + i1;
        const float x0 = __ldcg(w.X + (size_t)r0 * dm.d + f), x1 = __ldcg(w.X + (size_t)r1 * dm.d + f);
        float s0 = 0.f, s1 = 0.f;
#pragma unroll 1
        for (int k0 = 0; k0 < n; k0 += 6) {   // the sharing blocks (this one included), six at a time
          unsigned long long pw[2][6];
          const unsigned long long* src[6];
#pragma unroll
          for (int k = 0; k < 6; ++k) {
            const int c2 = c_first + min(k0 + k, n - 1);   // past the last one: it is read again and ignored
            src[k] = p.pbuf + ((size_t)(2 * c2 + (c2 == c_first ? 1 : 0)) * Rp + c0) * kTileN + fl;
          }
          for (uint32_t spin = 0;; ++spin) {
            bool ok = true;
#pragma unroll
            for (int k = 0; k < 6; ++k) {
              pw[0][k] = ld_relaxed_u64(src[k] + (size_t)i * kTileN);
              pw[1][k] = ld_relaxed_u64(src[k] + (size_t)i1 * kTileN);
            }
#pragma unroll
            for (int k = 0; k < 6; ++k) ok = ok && (pw[0][k] >> 32) == (tag >> 32) && (pw[1][k] >> 32) == (tag >> 32);
            if (ok) break;
            if (spin > 16) {
              if (*af) break;
              if ((spin & 63) == 0 && *reinterpret_cast<volatile int*>(p.abort_g)) { *af = 1; break; }
              if (spin > 4096) __nanosleep(64);
              if (spin >= kMegaSpin) {
                *af = 1;
                att_note_timeout(p.abort_g, 7, gseq);
                *reinterpret_cast<volatile int*>(p.abort_g) = 1;
                atomicCAS(w.status, DEV_OK, DEV_TIMEOUT);
                break;
              }
            }
          }
#pragma unroll
          for (int k = 0; k < 6; ++k) {
            const bool use = k0 + k < n;
            s0 += use ? __uint_as_float((unsigned)pw[0][k]) : 0.f;
            s1 += use ? __uint_as_float((unsigned)pw[1][k]) : 0.f;
          }
        }
        const float y0 = x0 + s0, y1 = x1 + s1;
        w.X[(size_t)r0 * dm.d + f] = y0;
        store_act<bf16>(w.A, R, dm.d, r0, f, y0 * gn);
        if (i1 != i) {
          w.X[(size_t)r1 * dm.d + f] = y1;
          store_act<bf16>(w.A, R, dm.d, r1, f, y1 * gn);
        }
        const float q0 = warp_sum(y0 * y0), q1 = warp_sum(y1 * y1);
        if (lane == 0) {
          ctl->red[grp][quarter][i] = q0;
          ctl->red[grp][quarter][i1] = q1;
        }
      }
      bar_sync(bar_id, 128);
      if (et >= a && et < b)
        p.sumsq[((size_t)buf * nt128 + tile) * kMegaMaxRows + c0 + et] =
            ctl->red[grp][0][et] + ctl->red[grp][1][et] + ctl->red[grp][2][et] + ctl->red[grp][3][et];
      bar_sync(bar_id, 128);
    }
  }
  if (et == 0) MEGA_EV(sidx, 6);
}

// a1 + first a2: embedding gather, fp32 residual stream, first GEMM input planes, sums of squares, and
// this step's rotary table.  All 256 workers.
__device__ __forceinline__ void mega_embed(MegaCtl* ctl, const MegaParams& p, const StepArgs* __restrict__ args,
                                           const KvView& kv, const Work& w, const Dims& dm, int wt) {
  const int ww = wt >> 5, lane = wt & 31, R = p.R, nt = dm.d / kTileN, gamma = p.rows - 1;
  for (int item = blockIdx.x * 8 + ww; item < R * nt; item += gridDim.x * 8) {
    const int r = item / nt, tile = item % nt, b = ctl->row_b[r], j = ctl->row_j[r];
    const int seq = args->seq_ids[b];
    int tok = (j == 0) ? kv.pending[seq] : args->draft_ids[b * gamma + j - 1];
    tok = min(max(tok, 0), dm.V - 1);
    const int f = tile * kTileN + lane * 4;
    const uint2 raw = *reinterpret_cast<const uint2*>(p.embed + (size_t)tok * dm.d + f);
    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
    const float2 a = __bfloat1622float2(h2[0]), c2 = __bfloat1622float2(h2[1]);
    const float x[4] = {a.x, a.y, c2.x, c2.y};
    *reinterpret_cast<float4*>(w.X + (size_t)r * dm.d + f) = make_float4(x[0], x[1], x[2], x[3]);
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      store_act<bf16>(w.A, R, dm.d, r, f + i, x[i] * __bfloat162float(p.gain0[f + i]));
      ss += x[i] * x[i];
    }
    ss = warp_sum(ss);
    if (lane == 0) p.sumsq[(size_t)tile * kMegaMaxRows + r] = ss;
  }
  const int half = dm.hd / 2;
  for (int idx = blockIdx.x * kMegaWorkers + wt; idx < R * half; idx += gridDim.x * kMegaWorkers) {
    const int r = idx / half, i = idx % half;
    const int pos = ctl->plan.L[ctl->row_b[r]] + ctl->row_j[r];
    double s, c;
    sincos((double)pos * w.inv_freq[i], &s, &c);
    w.rope[idx] = make_float2((float)c, (float)s);
  }
}

// a10 tail + a11..a15 for sequence b = blockIdx.x (256 workers, named barrier 1).
__device__ __forceinline__ void mega_finalize(MegaCtl* ctl, const MegaParams& p, const StepArgs* __restrict__ args,
                                              const KvView& kv, const Work& w, const Dims& dm, int wt) {
  const int b = blockIdx.x, gamma = p.rows - 1, rows = p.rows, R = p.R;
  const int lane = wt & 31, warp = wt >> 5, nwarp = kMegaWorkers >> 5;
  const int seq = args->seq_ids[b];
  const int n_vtiles = (dm.V + kTileN - 1) / kTileN, nt128 = dm.d / kTileN;
  const bf16* gainF = p.lp[p.l1 - 1].gain_next;
  for (int j = 0; j < rows; ++j) {
    const int r = b * rows + j;
    RowStat a; a.m = -INFINITY; a.s = 0.f; a.arg = 0; a.pad = 0;
    const int per = (n_vtiles + kMegaWorkers - 1) / kMegaWorkers;
    const int t0 = wt * per, t1 = min(t0 + per, n_vtiles);
    for (int t = t0; t < t1; ++t) {
      RowStat x;
      const float4 raw = __ldcg(reinterpret_cast<const float4*>(w.stats + (size_t)t * R + r));
      x.m = raw.x; x.s = raw.y; x.arg = __float_as_int(raw.z); x.pad = __float_as_int(raw.w);
      a = stat_merge(a, x);
    }
    ctl->u.sred[wt] = a;
    bar_sync(1, kMegaWorkers);
    for (int stride = 1; stride < kMegaWorkers; stride <<= 1) {
      if ((wt % (2 * stride)) == 0 && wt + stride < kMegaWorkers)
        ctl->u.sred[wt] = stat_merge(ctl->u.sred[wt], ctl->u.sred[wt + stride]);
      bar_sync(1, kMegaWorkers);
    }
    if (wt == 0) { ctl->rs[j] = ctl->u.sred[0]; w.rowstat[r] = ctl->u.sred[0]; }
    bar_sync(1, kMegaWorkers);
  }
  // 1/rms of the final norm for this sequence's rows
  if (wt < rows) {
    float s = 0.f;
    for (int t = 0; t < nt128; ++t) s += __ldcg(p.sumsq + (size_t)t * kMegaMaxRows + b * rows + wt);
    ctl->inv[b * rows + wt] = 1.0f / sqrtf(s / (float)dm.d + dm.eps);
  }
  bar_sync(1, kMegaWorkers);
  if (args->dbg_hidden) {
    for (int idx = wt; idx < rows * dm.d; idx += kMegaWorkers) {
      const int r = b * rows + idx / dm.d, i = idx % dm.d;
      args->dbg_hidden[(size_t)r * dm.d + i] = __ldcg(w.X + (size_t)r * dm.d + i) * __bfloat162float(gainF[i]) * ctl->inv[r];
    }
  }
  for (int j = 1 + warp; j <= gamma; j += nwarp) {
    const int r = b * rows + j;
    float a = 0.f;
    if (args->has_judge)
      for (int i = lane; i < dm.d; i += 32)
        a = fmaf(__ldcg(w.X + (size_t)r * dm.d + i) * __bfloat162float(gainF[i]) * ctl->inv[r], w.judge_w[i], a);
    a = warp_sum(a);
    if (lane == 0) {
      const float s = args->has_judge ? 1.0f / (1.0f + expf(-(a + args->judge_bias))) : 0.f;
      ctl->score[j] = s;
      args->judge_scores[b * gamma + j - 1] = s;
    }
  }
  bar_sync(1, kMegaWorkers);
  if (warp == 0) {
    bool ok = true;
    if (lane < gamma) {
      const int j = lane + 1;
      const int d = args->draft_ids[b * gamma + lane];
      const RowStat st = ctl->rs[j - 1];
      const float zd = __ldcg(w.tgt_logit + b * rows + j - 1) - st.m;
      const float pr = expf(zd) / st.s;
      args->p_draft[b * gamma + lane] = pr;
      if (args->logp_draft) args->logp_draft[b * gamma + lane] = zd - logf(st.s);
      bool align;
      if (args->mode == 0) align = args->top_k >= 2 ? st.pad < args->top_k : (d == st.arg);
      else align = args->uniforms[b * rows + lane] * args->q_tok[b * gamma + lane] < pr;
      const bool judge = args->has_judge && (ctl->score[j] > args->theta[b]);
      ok = (args->use_align && align) || (args->use_judge && judge) || args->accept_all;
    }
    const unsigned rej = __ballot_sync(0xffffffffu, !ok);
    const int n = rej ? (__ffs(rej) - 1) : gamma;
    if (lane == 0) {
      const int L = ctl->plan.L[b];
      args->accepted_len[b] = n;
      args->new_kv_len[b] = L + 1 + n;
      if (args->mode == 0) {
        const int nxt = ctl->rs[n].arg;
        args->next_token[b] = nxt;
        if (args->commit) kv.pending[seq] = nxt;
      }
      if (args->commit) kv.kv_len[seq] = L + 1 + n;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
template <int HD, int SLOTS, bool kTr, bool A5>
__global__ void __launch_bounds__(kMegaThreads, 1)
k_verify_mega(const __grid_constant__ MegaMaps mp, const MegaParams p, const StepArgs* __restrict__ args, const KvView kv,
              const Work w, const Dims dm) {
  extern __shared__ uint8_t mega_smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(mega_smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* q_area = ring + (size_t)p.stages * p.stage_bytes;
  MegaCtl* ctl = reinterpret_cast<MegaCtl*>(q_area + p.q_area_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c = blockIdx.x, G = gridDim.x, NS = p.stages, B = p.B, R = p.R, Rp = p.Rp, rows = p.rows;
  AttGeom g = att_geom(HD, dm.Hq / dm.Hkv, rows);
  if constexpr (A5) { g.KPS = kA5Keys; g.KS = 1; g.KW = kA5Keys; }   // one sub-partial per block segment

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(smem_u32(&ctl->full[i]), 2);
      mbar_init(smem_u32(&ctl->empty[i]), 1);
      ctl->cons_cnt[i] = 0;
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&ctl->tmem_full[i]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[i]), kMegaWorkers);
      mbar_init(smem_u32(&ctl->a5.s_full[i]), 1);
      mbar_init(smem_u32(&ctl->a5.p_full[i]), 128);
      mbar_init(smem_u32(&ctl->a5.o_done[i]), 1);
      mbar_init(smem_u32(&ctl->a5_pair[i]), 64);
    }
    mbar_init(smem_u32(&ctl->a5.q_ready), 128);
    ctl->abort_flag = 0;
    ctl->bars_passed = 0;
    int acc = 0;
    for (int b = 0; b < B; ++b) {
      const int L = kv.kv_len[args->seq_ids[b]];
      ctl->plan.L[b] = L;
      ctl->plan.pre[b] = acc;
      acc += L > 0 ? dm.Hkv * ((L + g.KPS - 1) / g.KPS + (A5 ? kA5Pad : 0)) : 0;
    }
    ctl->plan.pre[B] = acc;
    ctl->plan.T = acc;
    ctl->plan.pad = A5 ? kA5Pad : 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"(p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x < R) {
    const int r = threadIdx.x, b = r / rows, j = r % rows, gamma = rows - 1;
    const int pos = ctl->plan.L[b] + j;
    ctl->row_b[r] = b;
    ctl->row_j[r] = j;
    ctl->row_page[r] = kv.block_table[(size_t)args->seq_ids[b] * kv.max_pages_per_seq + pos / kv.page_size];
    ctl->row_slot[r] = pos % kv.page_size;
    ctl->tgt_tok[r] = (j < gamma) ? args->draft_ids[b * gamma + j] : -1;
    ctl->row_qoff[r] = (b * dm.Hq * rows + j) * dm.hd;
    ctl->row_nkvoff[r] = (b * dm.Hkv * 2 * rows + j) * dm.hd;
    ctl->row_kvoff[r] = ((long long)ctl->row_page[r] * 2 * dm.Hkv * kv.page_size + ctl->row_slot[r]) * dm.hd;
  }
  __syncthreads();

  const AttPlan& pl = ctl->plan;
  const long long t_lo = (long long)c * pl.T / G, t_hi = (long long)(c + 1) * pl.T / G;
  // ring stages of one attention phase: one per tile, or (tcgen05) a key stage and a value stage per real tile
  int n_att = (int)(t_hi - t_lo);
  if constexpr (A5) {
    int n_real = 0;
    for (long long t = t_lo; t < t_hi;) {
      const AttTile x = att_locate(pl, B, g.KPS, (int)t);
      const int nv = (int)min((long long)(x.nt_b - x.ti), t_hi - t);
      n_real += max(0, min(nv, x.nt_real - x.ti));
      t += nv;
    }
    n_att = 2 * n_real;
  }
  const A5Ring a5r{ctl->full, ctl->empty, ring, p.stage_bytes, NS, &ctl->abort_flag, p.abort_g, w.status};
  att_fill_pages(ctl->att_pages, pl, kv, args, B, g.KPS, t_lo, t_hi, threadIdx.x, blockDim.x);
  __syncthreads();
  auto stage_addr = [&](int s) -> uint32_t { return smem_u32(ring + (size_t)s * p.stage_bytes); };

  // Register reallocation between warpgroups: the single-thread roles need few registers, the workers
  // (fused epilogues, attention fragments) many.  Under the 384-thread launch bound of 168 registers per
  // thread the workers spill, and with 227 KB of the SM's memory configured as shared memory a spill reload
  // rarely hits L1: it costs an L2 round trip.
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kMegaRegsLight));
  if (warp == 0) {
    // ------------------------------ weight / cache-tile producer ------------------------------
    // One lane; all 32 with the tcgen05 attention, whose cache tiles are 32 small copies each (one per lane, one
    // instruction per tile).  All lanes run the same control flow and wait on the same barriers; lane 0 alone announces
    // bytes and issues the weight copies.
    if (lane < (A5 ? 32 : 1)) {
      const uint64_t pol_w = l2_policy_evict_first();
      RingPos rp{0, 0, NS};
      int sidx = 0;
      bool alive = true;
      auto wait_slot = [&]() -> bool {
        return rp.r == 0 || mega_wait(smem_u32(&ctl->empty[rp.s]), (uint32_t)(rp.r - 1) & 1u, ctl, p, w.status, 1, rp.r);
      };
      auto fsite = [&](int site, int l) {
        if (!alive) return;
        const SiteSplit ss = site_split(site, dm, c, G);
        const int li = l - p.l0;
        const int tq = dm.Hq * dm.hd / kTileN, tk = dm.Hkv * dm.hd / kTileN;
        unsigned u = ss.g_lo;
        Seg sg;
        while (seg_next(ss, u, sg)) {
          // the tensor map(s) and row of this segment's tile; only the K coordinate changes per unit
          const CUtensorMap* tm0;
          const CUtensorMap* tm1 = nullptr;
          int row = sg.tile * kTileN;
          if (site == SITE_QKV) {
            if (sg.tile < tq) tm0 = &mp.wq[li];
            else if (sg.tile < tq + tk) { tm0 = &mp.wk[li]; row = (sg.tile - tq) * kTileN; }
            else { tm0 = &mp.wv[li]; row = (sg.tile - tq - tk) * kTileN; }
          } else if (site == SITE_O) tm0 = &mp.wo[li];
          else if (site == SITE_GU) { tm0 = &mp.wg[li]; tm1 = &mp.wu[li]; row = sg.tile * 64; }
          else if (site == SITE_DOWN) tm0 = &mp.wd[li];
          else tm0 = &mp.lm;
          for (int kb = sg.a; kb < sg.b; ++kb) {
            if (!wait_slot()) { alive = false; return; }
            if (lane == 0) {
              const uint32_t bar = smem_u32(&ctl->full[rp.s]), dst = stage_addr(rp.s);
              mbar_expect_tx(bar, kWTileBytes);
              tma_load_2d(dst, tm0, bar, kb * kBK, row, pol_w);
              if (site == SITE_GU) tma_load_2d(dst + 8192u, tm1, bar, kb * kBK, row, pol_w);
            }
            rp.next();
          }
        }
        if (lane == 0) MEGA_EV(sidx, 7);
        ++sidx;
      };
      auto fatt = [&](int l) {
        if (!alive) return;
        if constexpr (A5) {
          A5Pos ap{rp.s, rp.r};
          alive = a5_produce(a5r, ap, &mp.pool, kv, args, pl, B, l, t_lo, t_hi, ctl->att_pages, lane);
          rp.s = ap.s;
          rp.r = ap.r;
          return;
        }
        for (long long t = t_lo; t < t_hi; ++t) {
          if (!wait_slot()) { alive = false; return; }
          const uint32_t bar = smem_u32(&ctl->full[rp.s]);
          mbar_expect_tx(bar, kAttStageBytes);
          mbar_arrive(bar);   // stands in for the activation producer, which skips cache tiles
          const AttTile x = att_locate(pl, B, g.KPS, (int)t);
          const int ai = (int)(t - t_lo) * (g.KPS / 16);
          att_issue_tile(&mp.pool, kv, l, args->seq_ids[x.b], x.h, x.ti, x.L, g.KPS, HD, stage_addr(rp.s), bar,
                         ai + g.KPS / 16 <= kAttPageCache ? ctl->att_pages + ai : nullptr);
          rp.next();
        }
      };
      mega_walk(p, fsite, fatt);
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(2 * Rp);
      const uint32_t tmem_base = ctl->tmem_base;
      RingPos rp{0, 0, NS};
      int seg = 0, sidx = 0, nb = p.do_embed ? 1 : 0;
      bool alive = true;
      auto fsite = [&](int site, int l) {
        if (!alive) return;
        const SiteSplit ss = site_split(site, dm, c, G);
        bool first = true;
        unsigned u = ss.g_lo;
        // Do not look at this phase's stages before the phase has begun: the attention phase in between
        // may reuse a stage several times, and a parity wait started two uses early would be satisfied by
        // the wrong one.
        if (u < ss.g_hi && !mega_wait_bars(nb, ctl, p, w.status, 10)) { alive = false; return; }
        nb += (site == SITE_QKV) ? 3 : 1;
        Seg sg;
        while (seg_next(ss, u, sg)) {
          const int len = sg.b - sg.a;
          if (len == 0) continue;   // no share of this segment: no accumulator is used
          const int acc = seg & 1, use = seg >> 1;
          if (use > 0 && !mega_wait(smem_u32(&ctl->tmem_empty[acc]), (uint32_t)(use - 1) & 1u, ctl, p, w.status, 4, seg)) {
            alive = false;
            return;
          }
          tc_fence_after();
          const uint32_t dcol = tmem_base + (uint32_t)(acc * 2 * Rp);
          for (int i = 0; i < len; ++i) {
            if (!mega_wait(smem_u32(&ctl->full[rp.s]), (uint32_t)rp.r & 1u, ctl, p, w.status, 5, rp.r)) { alive = false; return; }
            tc_fence_after();
            if (first) { MEGA_EV(sidx, 2); first = false; }
            const uint32_t wa = stage_addr(rp.s);
            const uint64_t dw = smem_desc_sw128(wa), da = smem_desc_sw128(wa + kWTileBytes);
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k) tc_mma_bf16(dcol, dw + 2 * k, da + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
            tc_commit(smem_u32(&ctl->empty[rp.s]));
            rp.next();
          }
          tc_commit(smem_u32(&ctl->tmem_full[acc]));
          ++seg;
        }
        MEGA_EV(sidx, 3);
        ++sidx;
      };
      int a5_tiles = 0, a5_segs = 0;
      auto fatt = [&](int l) {
        if constexpr (A5) {
          if (!alive) return;
          A5Pos ap{rp.s, rp.r};
          alive = a5_issue(a5r, ap, &ctl->a5, tmem_base, smem_u32(q_area), g.nq, 0, pl, B, t_lo, t_hi, a5_tiles, a5_segs);
          rp.s = ap.s;
          rp.r = ap.r;
        } else {
          rp.advance(n_att);
        }
      };
      mega_walk(p, fsite, fatt);
    }
  } else {
    // ------------------------------ activation producers (warps 2 and 3) ------------------------------
    // Two threads, alternate units: right after a device-wide barrier the ring already holds the phase's first
    // weight tiles, and the MMAs can start only as fast as their activation slices are requested (a wait, an
    // expect and a TMA per slice cost one thread about a quarter of a microsecond).
    if (lane == 0) {
      const int mine = warp - 2;
      int n_unit = 0;
      const uint64_t pol_a = l2_policy_evict_last();
      const uint32_t a_tx = (uint32_t)(2 * Rp) * 128u;
      RingPos rp{0, 0, NS};
      int nb = p.do_embed ? 1 : 0, sidx = 0;
      bool alive = true;
      auto fsite = [&](int site, int l) {
        if (!alive) return;
        const SiteSplit ss = site_split(site, dm, c, G);
        if (ss.g_hi > ss.g_lo) {
          // inputs of this phase are complete once `nb` device-wide barriers have been passed
          if (!mega_wait_bars(nb, ctl, p, w.status, 3)) { alive = false; return; }
          __threadfence();
          fence_proxy_async();
          if (mine == 0) MEGA_EV(sidx, 0);
          const CUtensorMap* tm = (site == SITE_O) ? &mp.a_q : (site == SITE_DOWN ? &mp.a_f : &mp.a_d);
          unsigned u = ss.g_lo;
          Seg sg;
          while (seg_next(ss, u, sg)) {
            for (int kb = sg.a; kb < sg.b; ++kb, ++n_unit) {
              if ((n_unit & 1) == mine) {
                if (rp.r > 0 && !mega_wait(smem_u32(&ctl->empty[rp.s]), (uint32_t)(rp.r - 1) & 1u, ctl, p, w.status, 2, rp.r)) {
                  alive = false;
                  return;
                }
                const uint32_t bar = smem_u32(&ctl->full[rp.s]);
                mbar_expect_tx(bar, a_tx);
                tma_load_2d(stage_addr(rp.s) + kWTileBytes, tm, bar, kb * kBK, 0, pol_a);
              }
              rp.next();
            }
          }
          if (mine == 0) MEGA_EV(sidx, 1);
        }
        ++sidx;
        nb += (site == SITE_QKV) ? 3 : 1;
      };
      int a5_tiles = 0, a5_segs = 0;
      auto fatt = [&](int l) {
        if constexpr (A5) {
          // warp 2 issues the attention MMAs of the odd tiles (warp 1 those of the even ones)
          if (mine == 0) {
            if (!alive) return;
            A5Pos ap{rp.s, rp.r};
            alive = a5_issue(a5r, ap, &ctl->a5, ctl->tmem_base, smem_u32(q_area), g.nq, 1, pl, B, t_lo, t_hi, a5_tiles, a5_segs);
            rp.s = ap.s;
            rp.r = ap.r;
            return;
          }
        }
        rp.advance(n_att);
      };
      mega_walk(p, fsite, fatt);
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kMegaRegsHeavy));
    // ------------------------------ workers ------------------------------
    const int wt = threadIdx.x - 128, ww = wt >> 5;
    int nbar = 0, gseq = 0, seg = 0, it = 0;
    int a5_tiles = 0, a5_pairs = 0;
    bool alive = true;
    if (p.do_embed) {
      mega_embed(ctl, p, args, kv, w, dm, wt);
      alive = mega_grid_sync<kTr>(ctl, p, w.status, nbar, wt);
    }
    auto units = [&](int site) -> int { return site_units(site_split(site, dm, c, G)); };
    auto gemm_phase = [&](int site, int l) {
      ++gseq;
      if (alive) mega_epilogue<HD, SLOTS, kTr>(site, l, gseq, seg, ctl, p, args, kv, w, dm, wt);
      it += units(site);
      alive = mega_grid_sync<kTr>(ctl, p, w.status, nbar, wt);
    };
    const int n_ph = mega_n_phases(p);
    for (int ph = 0; ph < n_ph; ++ph) {
      int site, l;
      mega_phase(p, ph, site, l);
      if (site >= 0) {
        gemm_phase(site, l);
        continue;
      }
      // attention over the cache tiles of the ring, then the combine
      if (alive) {
        // attention events of the traced block go to the second event set of the layer's QKV phase
        unsigned long long* ev = (kTr && p.trace && c == (int)p.trace_block && (l - p.l0) * 4 < kMegaTraceSites)
                                     ? p.trace + 2 * kMegaTraceBarriers + 8 * kMegaTraceSites + (size_t)(l - p.l0) * 4 * 8
                                     : nullptr;
        AttRing rg{ctl->full, ctl->empty, ctl->cons_cnt, ring, p.stage_bytes, NS, &ctl->abort_flag, p.abort_g, w.status, ev};
        AttArgs aa{w.Qb, l < p.att_precise_layers ? w.Qlo : nullptr, w.KVn, AttPartials{w.tc_m, w.tc_l, w.tc_o}, p.n_tail_base, l};
        if constexpr (A5) {
          if ((ww & 3) < 2) {
            // softmax warps: lane quarter ww & 3, key / dim half ww >> 2
            alive = a5_softmax(a5r, &ctl->a5, ctl->tmem_base, q_area, &ctl->u.a5_mx[0][0][0], &ctl->a5_pair[ww & 3], a5_pairs, aa, pl, B,
                               dm.Hkv, g.nq, t_lo, t_hi, a5_tiles, c, ww & 3, ww >> 2, lane, ev);
          } else {
            // the other four warps: the causal tails (one m-tile of one (sequence, KV head) per task), dealt over
            // all blocks from the last block down
            AttWarp<HD, 2> st;
            const int k = (ww & 1) + 2 * (ww >> 2);
            for (int q = (G - 1 - c) * 4 + k; q < B * dm.Hkv * g.MT; q += G * 4)
              att_tail_task<HD, 2>(st, g, aa, q / g.MT, (q % g.MT) * 16, lane);
          }
        } else {
          int it2 = it;
          att_consume_dispatch<HD>(rg, it2, pl, g, args, kv, aa, dm.Hkv, c, G, ww, lane);
        }
      }
      it += n_att;
      alive = mega_grid_sync<kTr>(ctl, p, w.status, nbar, wt);
      if (alive) {
        const AttPartials P{w.tc_m, w.tc_l, w.tc_o};
        const int items = B * dm.Hkv * g.nq * AttCombineSplit<HD>::value;
        for (int item = ww * G + c; item < items; item += G * 8)   // spread over blocks first
          att_combine_item<bf16, HD, A5 ? 8 : 0>(P, pl, g, G, p.n_tail_base, dm.Hkv, item, w.ATT, R, dm.Hq, lane,
                                     (kTr && p.trace && c == 0 && ww == 0 && (l - p.l0) * 4 < kMegaTraceSites)
                                         ? p.trace + 2 * kMegaTraceBarriers + 8 * kMegaTraceSites + (size_t)(l - p.l0) * 4 * 8 + 4
                                         : nullptr);
      }
      alive = mega_grid_sync<kTr>(ctl, p, w.status, nbar, wt);
    }
    if (p.do_lm && alive && c < B) mega_finalize(ctl, p, args, kv, w, dm, wt);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    if (*reinterpret_cast<volatile int*>(&ctl->abort_flag)) __nanosleep(20000);   // let copies in flight land
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(ctl->tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

}  // namespace sj
