// Attention of the verification step on the 5th-generation tensor cores (head dimension 128, bf16 cache):
// the cached keys of the multi-kernel path, split along the keys over all SMs like sj_attn_tc.cuh's kernel,
// but with both contractions on tcgen05.mma and the scores in tensor memory.
//
// One work tile is 128 cached keys of one (sequence, KV head): K and V of its 8 pages arrive by TMA (boxes of
// 16 slots x 64 dims, 128-byte swizzle) as two 32 KiB shared-memory tiles laid out [half of the head dim][page]
// [16 keys x 128 B], so that the 128 key rows of a half sit 128 bytes apart.
//   S = Q K^T   M = 128 query-row slots (the group's gamma+1 rows of every query head; unused slots are zero),
//               N = 128 keys, K = head dim: Q from shared memory (K-major), the key tile as a K-major B operand.
//               The cache is bf16, and both operands of an MMA have one type, so a query enters as the sum of two
//               bf16 terms (hi + lo, 16 significant bits): two MMAs per 16-dim step into the same accumulator.
//   softmax     one thread per query-row slot reads its row of S from tensor memory into registers (no cross-lane
//               traffic), keeps a stabiliser m (raised only when the row maximum exceeds it by more than 8 in the
//               log2 domain: then the thread rescales its row of O), and writes P = exp2(S - m) over the scores it
//               has just read, as two bf16 terms per 32-key chunk ([hi 16 columns | lo 16 columns]).  S is double-
//               buffered, so the next tile's scores are computed while this tile's P V runs.
//   O += P V    (two accumulators, one for the even and one for the odd tiles: each has its own issuing thread; they are
//               added when the segment ends)  A = P from tensor memory (M = 128 slots, K = 16 keys per step = one page), B = the page's V rows
//               as an MN-major operand (the head dim is the contiguous one: leading byte offset = the 16 KiB
//               between the two halves, stride byte offset = the 1 KiB between 8-key groups), N = head dim.
// A segment (the block's run of tiles of one (sequence, KV head)) ends with the unnormalised partial (m, l, o)
// per query row, in the format of sj_attn_tc.cuh, whose combine pass merges them; the block's own gamma+1 rows
// (the causal tail) are handled with that file's mma.sync routine.
//
// Roles (384 threads): warp 0 TMA producer of the key tiles, warp 11 of the value tiles (sixteen lanes each), warps 1
// and 10 issue the MMAs of the even and the odd tiles (warp 1 owns tensor memory: S twice, O twice = all 512 columns),
// warps 2..9 softmax (two threads per query row, TMEM lane quarter = warp % 4) and, after their tiles, the causal tails.
// Every wait is bounded.
#pragma once

#include "sj_attn_tc.cuh"
#include "sj_gemm_tc.cuh"

namespace sj {

constexpr int kT5Keys = 128;               // keys per tile
constexpr int kT5Pad = 5;                  // empty tiles the plan counts per (sequence, KV head): what a segment costs a block beyond its tiles
constexpr int kT5Threads = 384;
constexpr int kT5TileBytes = 32768;        // one K or V tile: 2 halves x 8 pages x 2 KiB
constexpr int kT5SmemBytes = 2 * kT5TileBytes /* Q hi, lo */ + 4 * kT5TileBytes /* K, V double-buffered */;

struct T5Ctl {
  uint64_t kfull[2], kempty[2], vfull[2], vempty[2], s_full[2], p_full[2], o_done[2], q_ready;
  uint64_t pair[4];      // the two softmax warps of a lane quarter (64 arrivals)
  uint32_t tmem_base;
  int abort_flag;
  float mx[2][2][128];   // [tile parity][key half][query-row slot]: row maxima (and, at a segment's end, sums) of the two threads of a row
  AttPlan plan;
  int pages[kAttPageCache];
};

__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,"
      "%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_ld32_nowait(uint32_t taddr, float* v) {   // results valid after tc_wait_ld()
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,"
      "%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]), "=f"(v[9]),
        "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15]), "=f"(v[16]), "=f"(v[17]), "=f"(v[18]),
        "=f"(v[19]), "=f"(v[20]), "=f"(v[21]), "=f"(v[22]), "=f"(v[23]), "=f"(v[24]), "=f"(v[25]), "=f"(v[26]), "=f"(v[27]),
        "=f"(v[28]), "=f"(v[29]), "=f"(v[30]), "=f"(v[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tc_st32f(uint32_t taddr, const float* v) {
  uint32_t r[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(v[i]);
  tc_st16(taddr, r);
  tc_st16(taddr + 16, r + 16);
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory descriptor of an MN-major operand in the [half][page][16 x 128 B] layout: 16 keys (one page) by
// 128 dims; the two 64-dim halves are `half_stride` bytes apart, the two 8-key groups 1024 bytes.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t saddr, uint32_t half_stride) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)((half_stride >> 4) & 0x3FFF) << 16;   // leading byte offset: along the contiguous (head) dimension
  d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset: along the keys
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// bf16 x bf16 -> fp32, M = 128, N = n; b_mn: the B operand is MN-major
__device__ __forceinline__ uint32_t instr_desc_bf16_mn(int n, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// byte offset of (row, dim) in a K-major tile of two [rows x 128 B] halves 16 KiB apart, 128-byte swizzle
__device__ __forceinline__ uint32_t t5_q_off(int row, int dim) {
  const int h = dim >> 6, c = (dim & 63) >> 3;
  return (uint32_t)(h * 16384 + row * 128 + ((c ^ (row & 7)) << 4) + (dim & 7) * 2);
}
// TMEM lane of query row q: the rows are dealt round-robin to the four lane quarters (one softmax warp each)
__device__ __forceinline__ int t5_lane_of_row(int q) { return 32 * (q & 3) + (q >> 2); }

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ bool t5_wait(uint64_t* bar, uint32_t parity, T5Ctl* ctl, int* status, int where) {
  return att_mbar_wait(att_smem_u32(bar), parity, &ctl->abort_flag, status, nullptr, where, 0);
}

__global__ void __launch_bounds__(kT5Threads, 1)
k_attn_t5(const __grid_constant__ CUtensorMap tmKV, const StepArgs* __restrict__ args, KvView kv, Work w, Dims dm, AttArgs a) {
  constexpr int HD = 128;
  extern __shared__ uint8_t t5_smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(t5_smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t *sQ = sm, *sK = sm + 2 * kT5TileBytes, *sV = sm + 4 * kT5TileBytes;
  T5Ctl* ctl = reinterpret_cast<T5Ctl*>(sm + kT5SmemBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_wait();
  pdl_launch();
  const int B = args->B, rows = args->gamma + 1, Hkv = dm.Hkv, group = dm.Hq / dm.Hkv, nq = group * rows;
  const int G = gridDim.x, c = blockIdx.x;
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      att_mbar_init(att_smem_u32(&ctl->kfull[i]), 1);
      att_mbar_init(att_smem_u32(&ctl->kempty[i]), 1);
      att_mbar_init(att_smem_u32(&ctl->vfull[i]), 1);
      att_mbar_init(att_smem_u32(&ctl->vempty[i]), 1);
      att_mbar_init(att_smem_u32(&ctl->s_full[i]), 1);
      att_mbar_init(att_smem_u32(&ctl->p_full[i]), 256);
      att_mbar_init(att_smem_u32(&ctl->o_done[i]), 1);
    }
    att_mbar_init(att_smem_u32(&ctl->q_ready), 256);
    for (int i = 0; i < 4; ++i) att_mbar_init(att_smem_u32(&ctl->pair[i]), 64);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) att_plan_fill(&ctl->plan, w.row_pos, B, rows, Hkv, kT5Keys, lane, kT5Pad);
  // unused query-row slots stay zero for the whole kernel
  for (int i = threadIdx.x; i < 2 * kT5TileBytes / 16; i += blockDim.x) reinterpret_cast<uint4*>(sQ)[i] = make_uint4(0, 0, 0, 0);
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(att_smem_u32(&ctl->tmem_base)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const AttPlan& pl = ctl->plan;
  const long long t_lo = (long long)c * pl.T / G, t_hi = (long long)(c + 1) * pl.T / G;
  att_fill_pages(ctl->pages, pl, kv, args, B, kT5Keys, t_lo, t_hi, threadIdx.x, blockDim.x);
  __syncthreads();
  const uint32_t tmem = ctl->tmem_base;   // columns: [0,256) S twice (P overwrites S in place), [256,512) O twice (one per issuer)
  volatile int* abort_flag = &ctl->abort_flag;

  if (warp == 0 || warp == 11) {
    // ------------------------------ TMA producers: warp 0 the key tiles, warp 11 the value tiles ------------------------------
    // Two warps, so that the key tiles, which the scores need first, never queue behind a value stage that is still
    // waiting for its P V.  A tile is sixteen boxes of 2 KiB (16 keys x 64 dims: a page's slots, one swizzle span
    // wide) and one thread gets a copy out only every 200 clocks or so: sixteen lanes issue one box each (half =
    // lane / 8, page = lane % 8), all in the same flow; lane 0 announces the bytes.
    if (lane < 16) {
      const int which = warp == 0 ? 0 : 1, half = lane >> 3, p = lane & 7;
      uint64_t* full = which ? ctl->vfull : ctl->kfull;
      uint64_t* empty = which ? ctl->vempty : ctl->kempty;
      uint8_t* base = which ? sV : sK;
      int g = 0;   // real tiles so far
      for (long long t = t_lo; t < t_hi; ++t) {
        const AttTile x = att_locate(pl, B, kT5Keys, (int)t);
        if (x.ti >= x.nt_real) continue;   // one of the plan's empty tiles
        const int st = g & 1, seq = args->seq_ids[x.b], last_page = (x.L - 1) / 16, tb = (int)(t - t_lo);
        int pi = x.ti * 8 + p;
        if (pi > last_page) pi = last_page;   // keys there are masked; reload a valid page
        const int page = (tb + 1) * 8 <= kAttPageCache ? ctl->pages[tb * 8 + p]
                                                       : __ldg(kv.block_table + (size_t)seq * kv.max_pages_per_seq + pi);
        const long long row = ((((long long)a.layer * kv.n_pages + page) * 2 + which) * kv.n_kv_heads + x.h) * 16;
        if (g >= 2 && !t5_wait(&empty[st], (uint32_t)((g >> 1) - 1) & 1u, ctl, w.status, 1)) break;
        const uint32_t bar = att_smem_u32(&full[st]);
        const uint32_t dst = att_smem_u32(base + (size_t)st * kT5TileBytes);
        if (lane == 0) att_mbar_expect_tx(bar, kT5TileBytes);
        att_tma_2d(dst + (uint32_t)(half * 16384 + p * 2048), &tmKV, bar, half * 64, (int)row);
        ++g;
      }
    }
  } else if (warp == 1 || warp == 10) {
    // ------------------------------ MMA issuers: warp 1 the even tiles, warp 10 the odd ones ------------------------------
    // One thread gets a tcgen05.mma out every 110 clocks or so whatever its shape, and a tile needs 16 for the scores
    // and 16 for the output; a second issuing thread doubles the rate.  The split is by tile parity: thread X owns
    // stage X of the key and value tiles, score buffer X and an output accumulator of its own (O_X; the two share the
    // rows' stabiliser and are added when the segment ends).  Within a thread the order is scores(g), output(g),
    // scores(g + 2): the tensor pipe executes one thread's MMAs in issue order, which is all the ordering the reuse of
    // score buffer X needs, and while the thread waits for the probabilities of its tile the other one issues.
    if (lane == 0) {
      const int X = warp == 1 ? 0 : 1;
      const uint32_t id_s = instr_desc_bf16_mn(kT5Keys, 0), id_o = instr_desc_bf16_mn(HD, 1);
      const uint64_t dq = smem_desc_sw128(att_smem_u32(sQ)), dql = smem_desc_sw128(att_smem_u32(sQ) + kT5TileBytes);
      const uint64_t dk = smem_desc_sw128(att_smem_u32(sK) + (uint32_t)X * kT5TileBytes);
      const uint64_t dv = smem_desc_mn_sw128(att_smem_u32(sV) + (uint32_t)X * kT5TileBytes, 16384u);
      const uint32_t d_s = tmem + (uint32_t)(X * 128), d_o = tmem + (uint32_t)(256 + X * 128);
      int it = 0, seg = 0;
      long long t = t_lo;
      bool alive = true;
      while (t < t_hi && alive) {
        const AttTile x = att_locate(pl, B, kT5Keys, (int)t);
        const int nv = (int)min((long long)(x.nt_b - x.ti), t_hi - t);   // with the plan's empty tiles
        const int n = max(0, min(nv, x.nt_real - x.ti));
        t += nv;
        if (n == 0) continue;   // only empty tiles of this (sequence, KV head): no segment
        bool first = true;
        // every segment's queries are waited for, also where this thread owns none of its tiles: a parity wait that
        // skipped a phase would be satisfied one phase early
        if (!t5_wait(&ctl->q_ready, (uint32_t)seg & 1u, ctl, w.status, 2)) break;
        for (int i = ((it & 1) == X) ? 0 : 1; i < n; i += 2) {
          const int g = it + i;
          const uint32_t par = (uint32_t)(g >> 1) & 1u;
          if (!t5_wait(&ctl->kfull[X], par, ctl, w.status, 3)) { alive = false; break; }
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) {
            const uint64_t off = (uint64_t)((k >> 2) * (16384 >> 4) + (k & 3) * 2);   // start-address field, 16-byte units
            tc_mma_bf16(d_s, dq + off, dk + off, id_s, k > 0 ? 1u : 0u);
            tc_mma_bf16(d_s, dql + off, dk + off, id_s, 1u);
          }
          tc_commit(att_smem_u32(&ctl->kempty[X]));
          tc_commit(att_smem_u32(&ctl->s_full[X]));
          if (!t5_wait(&ctl->p_full[X], par, ctl, w.status, 5) || !t5_wait(&ctl->vfull[X], par, ctl, w.status, 6)) { alive = false; break; }
          tc_fence_after();
#pragma unroll
          for (int pg = 0; pg < 8; ++pg) {   // the 16 keys of page pg: P's 32-column chunk pg / 2 holds [hi 16 | lo 16]
            const uint64_t db = dv + (uint64_t)(pg * (2048 >> 4));
            const uint32_t pa = d_s + (uint32_t)(32 * (pg >> 1) + 8 * (pg & 1));
            tc_mma_bf16_ta(d_o, pa, db, id_o, (!first || pg > 0) ? 1u : 0u);
            tc_mma_bf16_ta(d_o, pa + 16, db, id_o, 1u);
          }
          tc_commit(att_smem_u32(&ctl->vempty[X]));
          tc_commit(att_smem_u32(&ctl->o_done[X]));
          first = false;
        }
        it += n;
        ++seg;
      }
    }
  } else if (warp < 10) {
    // ------------------------------ softmax: two threads per query-row slot, 64 keys each ------------------------------
    // warps 2..5 take keys [0, 64) of every tile, warps 6..9 keys [64, 128); warp w reads TMEM lane quarter w % 4, so
    // warps w and w + 4 share a quarter: they exchange their row maxima through shared memory (a barrier of
    // their 64 threads) and keep separate sums, which are added when the segment's partial is written.
    const int half = (warp - 2) >> 2, quarter = warp & 3;
    const int sl = 32 * quarter + lane;                     // TMEM lane == query-row slot
    const int q = 4 * (sl & 31) + (sl >> 5);                // the query row of this slot (inverse of t5_lane_of_row)
    const bool active = q < nq;
    const uint32_t lane_addr = tmem + ((uint32_t)(32 * quarter) << 16);
    int it = 0, seg = 0, pair_n = 0;
    // hand-over between the quarter's two warps: a shared-memory barrier with a bounded wait, so that a warp that
    // gives up cannot strand its partner
    auto pair_sync = [&]() -> bool {
      att_mbar_arrive(att_smem_u32(&ctl->pair[quarter]));
      const bool ok = t5_wait(&ctl->pair[quarter], (uint32_t)pair_n & 1u, ctl, w.status, 10);
      ++pair_n;
      return __all_sync(0xffffffffu, ok);
    };
    // queries of a (sequence, KV head): fp16 (plus what its rounding dropped, in the two-term layers) -> two bf16 terms;
    // this thread converts its half of the head dimension (all loads first: one at a time they cost 0.4 us each)
    auto deliver_q = [&](const AttTile& x) {
      if (active) {
        const __half* qh = a.Qb + (((size_t)x.b * Hkv + x.h) * nq + q) * HD + 64 * half;
        const __half* ql = a.Qlo ? a.Qlo + (((size_t)x.b * Hkv + x.h) * nq + q) * HD + 64 * half : nullptr;
        uint4 raw[8], rawl[8];
#pragma unroll
        for (int d8 = 0; d8 < 8; ++d8) {
          raw[d8] = __ldcg(reinterpret_cast<const uint4*>(qh + 8 * d8));
          rawl[d8] = ql ? __ldcg(reinterpret_cast<const uint4*>(ql + 8 * d8)) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int d8 = 0; d8 < 8; ++d8) {
          const __half2* h2 = reinterpret_cast<const __half2*>(&raw[d8]);
          const __half2* l2 = reinterpret_cast<const __half2*>(&rawl[d8]);
          uint32_t hi[4], lo[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float2 v = __half22float2(h2[e]);
            const float2 vl = __half22float2(l2[e]);
            v.x += vl.x;
            v.y += vl.y;
            const __nv_bfloat162 bh = __floats2bfloat162_rn(v.x, v.y);
            const float2 back = __bfloat1622float2(bh);
            const __nv_bfloat162 bl = __floats2bfloat162_rn(v.x - back.x, v.y - back.y);
            hi[e] = *reinterpret_cast<const uint32_t*>(&bh);
            lo[e] = *reinterpret_cast<const uint32_t*>(&bl);
          }
          const uint32_t off = t5_q_off(sl, 64 * half + 8 * d8);
          *reinterpret_cast<uint4*>(sQ + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(sQ + kT5TileBytes + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMAs read these generic-proxy stores
      att_mbar_arrive(att_smem_u32(&ctl->q_ready));
    };
    long long t = t_lo;
    bool alive = true;
    // the block's next run of real tiles at or after tile t: (sequence, KV head, first tile), its length n, and nv,
    // the same with the plan's empty tiles; n == 0 when only empty tiles are left of that (sequence, KV head)
    auto run_at = [&](long long t, AttTile& x, int& n, int& nv) {
      x = att_locate(pl, B, kT5Keys, (int)t);
      nv = (int)min((long long)(x.nt_b - x.ti), t_hi - t);
      n = max(0, min(nv, x.nt_real - x.ti));
    };
    while (t < t_hi && alive) {
      AttTile x;
      int n, nv;
      run_at(t, x, n, nv);
      if (n == 0) {
        // only empty tiles of this (sequence, KV head) fell to this block: the combine pass still reads the block's
        // slot for it, so it gets a partial of weight zero (the stored outputs are finite: old values or zeros)
        const size_t base = (((size_t)c + (size_t)x.b * Hkv + x.h) * kAttMaxSub + 0) * (size_t)nq;
        if (active && half == 0) { a.P.m[base + q] = -INFINITY; a.P.l[base + q] = 0.f; }
        t += nv;
        continue;
      }
      if (seg == 0) deliver_q(x);   // later segments' queries were delivered while the segment before them ended
      float m_used = -INFINITY, l_sum = 0.f;
      for (int i = 0; i < n && alive; ++i) {
        const int g = it + i, sb = g & 1;
        int ok = 1;
        if (lane == 0) ok = t5_wait(&ctl->s_full[sb], (uint32_t)(g >> 1) & 1u, ctl, w.status, 7) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) { alive = false; break; }
        att_mbar_try(att_smem_u32(&ctl->s_full[sb]), (uint32_t)(g >> 1) & 1u);   // every lane observes the completed phase
        tc_fence_after();
        const uint32_t s_addr = lane_addr + (uint32_t)(sb * 128 + 64 * half);
        const int n_valid = min(kT5Keys, x.L - (x.ti + i) * kT5Keys) - 64 * half;   // this thread's keys >= n_valid are masked
        float sc[64];
        tc_ld32_nowait(s_addr, sc);
        tc_ld32_nowait(s_addr + 32, sc + 32);
        tc_wait_ld();
        if (!active) {   // a row slot without a query holds whatever its lane computed: keep it from moving the stabiliser
#pragma unroll
          for (int j = 0; j < 64; ++j) sc[j] = 0.f;
        }
        if (n_valid < 64) {   // warp-uniform; only a sequence's last tile
#pragma unroll
          for (int j = 0; j < 64; ++j) sc[j] = (j < n_valid) ? sc[j] : -INFINITY;
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains: a single one is 64 dependent steps
#pragma unroll
        for (int j = 0; j < 64; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], sc[j]);
        float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        ctl->mx[g & 1][half][sl] = mx;
        if (!pair_sync()) { alive = false; break; }
        mx = fmaxf(mx, ctl->mx[g & 1][half ^ 1][sl]);
        // the stabiliser only moves when the maximum outgrows it by more than 8 (p stays below 256)
        float m_new = m_used, f = 1.f;
        if (m_used == -INFINITY) m_new = mx;
        else if (mx > m_used + 8.f) { m_new = mx; f = ex2_approx(m_used - m_new); }
        if (i > 0 && __any_sync(0xffffffffu, f != 1.f)) {
          // rescale this thread's half of its row of both output accumulators: the previous tile's, once its P V has
          // completed (this tile's cannot start before every thread has delivered its P), and, from the segment's third
          // tile on, this tile's own (its last P V completed before the scores just read were computed: same issuer)
          if (lane == 0) ok = t5_wait(&ctl->o_done[(g - 1) & 1], (uint32_t)((g - 1) >> 1) & 1u, ctl, w.status, 8) ? 1 : 0;
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) { alive = false; break; }
          att_mbar_try(att_smem_u32(&ctl->o_done[(g - 1) & 1]), (uint32_t)((g - 1) >> 1) & 1u);
          tc_fence_after();
#pragma unroll 1
          for (int k = 0; k < (i >= 2 ? 2 : 1); ++k) {
            const uint32_t o_addr = lane_addr + (uint32_t)(256 + 128 * ((g - 1 + k) & 1));
#pragma unroll 1
            for (int c0 = 64 * half; c0 < 64 * half + 64; c0 += 32) {
              float o[32];
              tc_ld32(o_addr + c0, o);
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] *= f;
              tc_st32f(o_addr + c0, o);
            }
          }
          tc_wait_st();
          l_sum *= f;
        }
        // probabilities as two bf16 terms, written over the scores: chunk of 32 keys -> [hi 16 columns | lo 16 columns];
        // hi = p truncated to bf16, lo = the rest rounded to bf16 (16 significant bits in all)
        float ls4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
          uint32_t hi[16], lo[16];
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const float p0 = ex2_approx(sc[c0 + j] - m_new), p1 = ex2_approx(sc[c0 + j + 1] - m_new);   // 0 for masked keys
            ls4[(j >> 1) & 3] += p0 + p1;
            const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
            hi[j >> 1] = __byte_perm(b0, b1, 0x7632);
            const __nv_bfloat162 bl = __floats2bfloat162_rn(p0 - __uint_as_float(b0 & 0xffff0000u), p1 - __uint_as_float(b1 & 0xffff0000u));
            lo[j >> 1] = *reinterpret_cast<const uint32_t*>(&bl);
          }
          tc_st16(s_addr + (uint32_t)c0, hi);
          tc_st16(s_addr + (uint32_t)c0 + 16, lo);
        }
        l_sum += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
        tc_wait_st();
        tc_fence_before();
        att_mbar_arrive(att_smem_u32(&ctl->p_full[sb]));
        m_used = m_new;
      }
      if (!alive) break;
      // The next segment's queries, before this one is wound up: every score MMA of this segment has completed (this
      // thread saw the scores of its last tile), so the query tiles are free, and the issuers start on the next
      // segment's scores while the partial below is read out (its first P V waits for probabilities that this thread
      // delivers only afterwards, so the output accumulators are not touched early).
      for (long long t2 = t + nv; t2 < t_hi;) {
        AttTile x2;
        int n2, nv2;
        run_at(t2, x2, n2, nv2);
        if (n2 > 0) { deliver_q(x2); break; }
        t2 += nv2;
      }
      // the segment's partial: wait for the last P V of either issuer, then (m, l, o) of every real query row
      {
        const int g = it + n - 1;
        int ok = 1;
        if (lane == 0)
          ok = (t5_wait(&ctl->o_done[g & 1], (uint32_t)(g >> 1) & 1u, ctl, w.status, 9) &&
                (n < 2 || t5_wait(&ctl->o_done[(g - 1) & 1], (uint32_t)((g - 1) >> 1) & 1u, ctl, w.status, 9))) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        att_mbar_try(att_smem_u32(&ctl->o_done[g & 1]), (uint32_t)(g >> 1) & 1u);
        if (n >= 2) att_mbar_try(att_smem_u32(&ctl->o_done[(g - 1) & 1]), (uint32_t)((g - 1) >> 1) & 1u);
        tc_fence_after();
        ctl->mx[(g + 1) & 1][half][sl] = l_sum;           // the buffer the last tile did not use
        if (!pair_sync()) break;
        const float l_tot = l_sum + ctl->mx[(g + 1) & 1][half ^ 1][sl];
        const size_t base = (((size_t)c + (size_t)x.b * Hkv + x.h) * kAttMaxSub + 0) * (size_t)nq;
        if (active && half == 0) { a.P.m[base + q] = m_used; a.P.l[base + q] = l_tot; }
#pragma unroll 1
        for (int c0 = 64 * half; c0 < 64 * half + 64; c0 += 32) {
          float o[32];
          tc_ld32(lane_addr + (uint32_t)(256 + 128 * (g & 1)) + c0, o);
          if (n >= 2) {   // the other issuer's accumulator holds the other half of the segment's tiles
            float o2[32];
            tc_ld32(lane_addr + (uint32_t)(256 + 128 * ((g - 1) & 1)) + c0, o2);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] += o2[j];
          }
          if (active) {
            float4* dst = reinterpret_cast<float4*>(a.P.o + (base + q) * HD + c0);
#pragma unroll
            for (int j = 0; j < 8; ++j) dst[j] = make_float4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
          }
        }
        tc_fence_before();
        if (!pair_sync()) break;   // the sums have been read before the next segment's first tile reuses the buffer
      }
      it += n;
      t += nv;
      ++seg;
    }
    // the causal tails (the step's own rows as keys; mma.sync): one m-tile of one (sequence, KV head) per task, dealt
    // over all blocks' softmax warps from the last block down
    if (alive) {
      const AttGeom g = att_geom(HD, group, rows);
      AttWarp<HD, 2> st;
      for (int task = (G - 1 - c) * 8 + (warp - 2); task < B * Hkv * g.MT; task += G * 8)
        att_tail_task<HD, 2>(st, g, a, task / g.MT, (task % g.MT) * 16, lane);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    if (*abort_flag) __nanosleep(20000);   // let copies in flight land before the block retires
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}


// =============================================================================================
// The same attention as phase routines of a kernel whose shared-memory ring also carries other traffic (the
// persistent step kernel), for at most 64 query rows per (sequence, KV head) and ring stages of at least 32 KiB.
//
// A 128-key tile is two ring entries, the key tile and then the value tile, one stage each ([half][page][16 keys x
// 128 B] as above; each stage has its own full / empty barrier).  Query row q sits in TMEM lane q and in row q of a
// query area of its own, which holds pad8(nq) rows per 64-dim half: the MMAs run at M = 128 all the same, their rows
// beyond the area read whatever shared memory follows it (the caller guarantees 16 KiB of its own allocation after the
// last half's base) and produce accumulator lanes nobody reads; so only the lane quarters 0 and 1 carry rows, and four
// warps run the softmax (two threads per row, 64 keys each).
//
// Two issuing threads, split by tile parity as in the kernel above: thread X owns score buffer X (columns
// [128 X, +128); the probabilities are written over it) and output accumulator X (columns [256 + 128 X, +128)), issues
// scores(g), output(g), scores(g + 2) in that order, and the softmax adds the two accumulators when the segment ends.
// All 512 columns alias whatever the kernel keeps there outside the attention phase.
// =============================================================================================
constexpr int kA5Keys = 128;
constexpr int kA5MaxRows = 64;
constexpr uint32_t kA5Part = 32768;   // bytes of a key tile or a value tile: the least a ring stage must hold
constexpr int kA5TmemCols = 512;
constexpr int kA5Pad = 3;   // empty tiles the plan counts per (sequence, KV head), see AttPlan::pad

struct A5Bars {
  uint64_t s_full[2];   // one arrival: issuer X's commit after the score MMAs
  uint64_t p_full[2];   // 128 arrivals: the softmax threads
  uint64_t o_done[2];   // one arrival: issuer X's commit after the output MMAs
  uint64_t q_ready;     // 128 arrivals
};
struct A5Ring {
  uint64_t* full;    // [stages], each completes on two arrivals (the expecting one and a second)
  uint64_t* empty;   // [stages], one arrival
  uint8_t* base;
  int stage_stride, stages;
  volatile int* abort_flag;
  volatile int* abort_g;
  int* status;
};
struct A5Pos {
  int s, r;
  __device__ __forceinline__ void next(int NS) {
    if (++s == NS) { s = 0; ++r; }
  }
};
struct A5Entry {
  int s0, s1;
  uint32_t par0, par1, a0, a1;   // stage, parity of this use and address of the key tile (0) and the value tile (1)
};
__host__ __device__ __forceinline__ int a5_q_half_bytes(int nq) { return ((nq + 7) & ~7) * 128; }
__host__ __device__ __forceinline__ int a5_q_area_bytes(int nq) { return 4 * a5_q_half_bytes(nq); }   // two planes x two halves

__device__ __forceinline__ A5Entry a5_entry(const A5Ring& rg, A5Pos& pos) {   // the tile at pos; pos moves past it
  A5Entry e;
  e.s0 = pos.s;
  e.par0 = (uint32_t)pos.r & 1u;
  e.a0 = att_smem_u32(rg.base + (size_t)pos.s * rg.stage_stride);
  pos.next(rg.stages);
  e.s1 = pos.s;
  e.par1 = (uint32_t)pos.r & 1u;
  e.a1 = att_smem_u32(rg.base + (size_t)pos.s * rg.stage_stride);
  pos.next(rg.stages);
  return e;
}
__device__ __forceinline__ bool a5_wait(const A5Ring& rg, uint64_t* bar, uint32_t parity, int where, int extra) {
  return att_mbar_wait(att_smem_u32(bar), parity, rg.abort_flag, rg.status, rg.abort_g, where, extra);
}

// All 32 lanes of one warp (same control flow): the TMA loads of the block's tiles [t_lo, t_hi) of one layer.  A tile
// is sixteen boxes of 2 KiB for the keys and sixteen for the values (16 keys x 64 dims: a page's slots, one swizzle
// span wide), and one thread gets a copy out only every 200 clocks or so: every lane issues ONE box of each tile (lanes
// 0..15 keys, 16..31 values; half = lane / 8 % 2, page = lane % 8), so a tile costs one instruction.  Lane 0 announces
// the bytes.  pages: the block's page ids, eight per tile (clamped to the sequence's last page), for its first
// kAttPageCache / 8 tiles.
__device__ __forceinline__ bool a5_produce(const A5Ring& rg, A5Pos& pos, const CUtensorMap* tmKV, const KvView& kv,
                                           const StepArgs* __restrict__ args, const AttPlan& pl, int B, int layer,
                                           long long t_lo, long long t_hi, const int* pages, int lane) {
  const int which = lane >> 4, half = (lane >> 3) & 1, p = lane & 7;
  for (long long t = t_lo; t < t_hi; ++t) {
    const AttTile x = att_locate(pl, B, kA5Keys, (int)t);
    if (x.ti >= x.nt_real) continue;   // one of the plan's empty tiles: no ring entry
    const int seq = args->seq_ids[x.b], last_page = (x.L - 1) / 16, tb = (int)(t - t_lo);
    int pi = x.ti * 8 + p;
    if (pi > last_page) pi = last_page;   // keys there are masked; reload a valid page
    const int page = (tb + 1) * 8 <= kAttPageCache ? pages[tb * 8 + p]
                                                   : __ldg(kv.block_table + (size_t)seq * kv.max_pages_per_seq + pi);
    const long long row = ((((long long)layer * kv.n_pages + page) * 2 + which) * kv.n_kv_heads + x.h) * 16;
    // claim the key stage and the value stage: every lane waits (same flow), lane 0 announces
    uint32_t dst = 0, bar = 0;
    for (int st = 0; st < 2; ++st) {
      if (pos.r > 0 && !a5_wait(rg, &rg.empty[pos.s], (uint32_t)(pos.r - 1) & 1u, 1, pos.r)) return false;
      const uint32_t b_st = att_smem_u32(&rg.full[pos.s]);
      if (lane == 0) {
        att_mbar_expect_tx(b_st, kA5Part);
        att_mbar_arrive(b_st);   // the stage's second arrival
      }
      if (st == which) {
        bar = b_st;
        dst = att_smem_u32(rg.base + (size_t)pos.s * rg.stage_stride);
      }
      pos.next(rg.stages);
    }
    att_tma_2d(dst + (uint32_t)(half * 16384 + p * 2048), tmKV, bar, half * 64, (int)row);
  }
  return true;
}

// One thread per tile parity X: the score MMAs and the output MMAs of the block's tiles g with g % 2 == X.  gt: tiles of
// earlier layers (the barriers' phases run on across layers), segs: segments of earlier layers; both advanced.
__device__ __forceinline__ bool a5_issue(const A5Ring& rg, A5Pos& pos, A5Bars* ab, uint32_t tmem, uint32_t q_area, int nq, int X,
                                         const AttPlan& pl, int B, long long t_lo, long long t_hi, int& gt, int& segs) {
  const uint32_t id_s = instr_desc_bf16_mn(kA5Keys, 0), id_o = instr_desc_bf16_mn(128, 1);
  const uint32_t hs = (uint32_t)a5_q_half_bytes(nq);
  const uint64_t dq = smem_desc_sw128(q_area), dql = smem_desc_sw128(q_area + 2 * hs);
  const uint64_t q_half = (uint64_t)(hs >> 4), k_half = (uint64_t)(16384 >> 4);   // start-address field, 16-byte units
  const uint32_t d_s = tmem + (uint32_t)(128 * X), d_o = tmem + (uint32_t)(256 + 128 * X);
  long long t = t_lo;
  while (t < t_hi) {
    const AttTile x = att_locate(pl, B, kA5Keys, (int)t);
    const int nv = (int)min((long long)(x.nt_b - x.ti), t_hi - t);   // with the plan's empty tiles
    const int n = max(0, min(nv, x.nt_real - x.ti));
    t += nv;
    if (n == 0) continue;   // only empty tiles of this (sequence, KV head): no segment
    // every segment's queries are waited for, also where this thread owns none of its tiles: a parity wait that
    // skipped a phase would be satisfied one phase early
    if (!a5_wait(rg, &ab->q_ready, (uint32_t)segs & 1u, 2, segs)) return false;
    tc_fence_after();
    bool first = true;
    for (int i = 0; i < n; ++i) {
      const int g = gt + i;
      const A5Entry e = a5_entry(rg, pos);
      if ((g & 1) != X) continue;
      const uint32_t par = (uint32_t)(g >> 1) & 1u;
      if (!a5_wait(rg, &rg.full[e.s0], e.par0, 3, g)) return false;
      tc_fence_after();
      const uint64_t dk = smem_desc_sw128(e.a0);
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint64_t ko = (uint64_t)(k >> 2) * k_half + (uint64_t)(2 * (k & 3)), qo = (uint64_t)(k >> 2) * q_half + (uint64_t)(2 * (k & 3));
        tc_mma_bf16(d_s, dq + qo, dk + ko, id_s, k > 0 ? 1u : 0u);
        tc_mma_bf16(d_s, dql + qo, dk + ko, id_s, 1u);
      }
      tc_commit(att_smem_u32(&rg.empty[e.s0]));
      tc_commit(att_smem_u32(&ab->s_full[X]));
      if (!a5_wait(rg, &ab->p_full[X], par, 5, g) || !a5_wait(rg, &rg.full[e.s1], e.par1, 6, g)) return false;
      tc_fence_after();
      const uint64_t dv = smem_desc_mn_sw128(e.a1, 16384u);
#pragma unroll
      for (int pg = 0; pg < 8; ++pg) {   // the 16 keys of page pg: P's 32-column chunk pg / 2 holds [hi 16 | lo 16]
        const uint64_t db = dv + (uint64_t)(pg * (2048 >> 4));
        const uint32_t pa = d_s + (uint32_t)(32 * (pg >> 1) + 8 * (pg & 1));
        tc_mma_bf16_ta(d_o, pa, db, id_o, (!first || pg > 0) ? 1u : 0u);
        tc_mma_bf16_ta(d_o, pa + 16, db, id_o, 1u);
      }
      tc_commit(att_smem_u32(&rg.empty[e.s1]));
      tc_commit(att_smem_u32(&ab->o_done[X]));
      first = false;
    }
    gt += n;
    ++segs;
  }
  return true;
}

// byte offset of (row, dim) in one plane of the query area (two K-major halves `hs` bytes apart, 128-byte swizzle)
__device__ __forceinline__ uint32_t a5_q_off(int row, int dim, uint32_t hs) {
  return (uint32_t)(dim >> 6) * hs + (uint32_t)(row * 128 + ((((dim & 63) >> 3) ^ (row & 7)) << 4) + (dim & 7) * 2);
}

// The softmax side: four warps, two threads per query row.  quarter (0, 1): the TMEM lane quarter == rows
// [32 * quarter, +32); half (0, 1): keys [64 * half, +64) of every tile and dims [64 * half, +64) of the row's queries
// and output.  mx: [2][2][64] floats of shared memory; pair_bar: a shared-memory barrier of the quarter's 64 threads
// (count 64; every wait is bounded, so a warp that gives up cannot strand its partner), pair_n: its phases so far.
// slot0: the partial slot of the block's segment is slot0 + b * Hkv + h (sub-partial 0).
// ev: optional timeline of the block's last segment (global-timer ns), stamped by the first softmax warp:
// [0] queries delivered, [1] last tile's probabilities delivered, [2] partial stored, [3] first scores seen.
__device__ __forceinline__ bool a5_softmax(const A5Ring& rg, A5Bars* ab, uint32_t tmem, uint8_t* q_area, float* mx, uint64_t* pair_bar,
                                           int& pair_n, const AttArgs& a, const AttPlan& pl, int B, int Hkv, int nq, long long t_lo,
                                           long long t_hi, int& gt, int slot0, int quarter, int half, int lane,
                                           unsigned long long* ev = nullptr) {
  constexpr int HD = 128;
  const bool stamp = ev && quarter == 0 && half == 0 && lane == 0;
  const int q = 32 * quarter + lane;   // query row == TMEM lane == row of the query area
  const bool active = q < nq;
  const uint32_t hs = (uint32_t)a5_q_half_bytes(nq);
  const uint32_t lane_addr = tmem + ((uint32_t)(32 * quarter) << 16);
  float* mx_own = mx + half * 64 + q;
  float* mx_other = mx + (half ^ 1) * 64 + q;   // + 128 * (tile parity)
  auto pair_sync = [&]() -> bool {
    att_mbar_arrive(att_smem_u32(pair_bar));
    const bool ok = a5_wait(rg, pair_bar, (uint32_t)pair_n & 1u, 10, pair_n);
    ++pair_n;
    return __all_sync(0xffffffffu, ok);
  };
  // queries of a (sequence, KV head): fp16 (plus what its rounding dropped, in the two-term layers) -> two bf16 terms;
  // this thread converts its half of the head dimension (all loads first)
  auto deliver_q = [&](const AttTile& x) {
    if (active) {
      const __half* qh = a.Qb + (((size_t)x.b * Hkv + x.h) * nq + q) * HD + 64 * half;
      const __half* ql = a.Qlo ? a.Qlo + (((size_t)x.b * Hkv + x.h) * nq + q) * HD + 64 * half : nullptr;
      uint4 raw[8], rawl[8];
#pragma unroll
      for (int d8 = 0; d8 < 8; ++d8) {
        raw[d8] = __ldcg(reinterpret_cast<const uint4*>(qh + 8 * d8));
        rawl[d8] = ql ? __ldcg(reinterpret_cast<const uint4*>(ql + 8 * d8)) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int d8 = 0; d8 < 8; ++d8) {
        const __half2* h2 = reinterpret_cast<const __half2*>(&raw[d8]);
        const __half2* l2 = reinterpret_cast<const __half2*>(&rawl[d8]);
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float2 v = __half22float2(h2[e]);
          const float2 vl = __half22float2(l2[e]);
          v.x += vl.x;
          v.y += vl.y;
          const __nv_bfloat162 bh = __floats2bfloat162_rn(v.x, v.y);
          const float2 back = __bfloat1622float2(bh);
          const __nv_bfloat162 bl = __floats2bfloat162_rn(v.x - back.x, v.y - back.y);
          hi[e] = *reinterpret_cast<const uint32_t*>(&bh);
          lo[e] = *reinterpret_cast<const uint32_t*>(&bl);
        }
        const uint32_t off = a5_q_off(q, 64 * half + 8 * d8, hs);
        *reinterpret_cast<uint4*>(q_area + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(q_area + 2 * hs + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMAs read these generic-proxy stores
    att_mbar_arrive(att_smem_u32(&ab->q_ready));
  };
  // the block's run of real tiles at tile t: (sequence, KV head, first tile), its length n, and nv, the same with the
  // plan's empty tiles; n == 0 when only empty tiles of that (sequence, KV head) fell to this block
  auto run_at = [&](long long t, AttTile& x, int& n, int& nv) {
    x = att_locate(pl, B, kA5Keys, (int)t);
    nv = (int)min((long long)(x.nt_b - x.ti), t_hi - t);
    n = max(0, min(nv, x.nt_real - x.ti));
  };
  long long t = t_lo;
  bool first_seg = true;
  while (t < t_hi) {
    AttTile x;
    int n, nv;
    run_at(t, x, n, nv);
    if (n == 0) {
      // the combine pass still reads the block's slot for this (sequence, KV head): a partial of weight zero (the
      // stored outputs are finite: old values or zeros)
      const size_t base = (((size_t)slot0 + (size_t)x.b * Hkv + x.h) * kAttMaxSub + 0) * (size_t)nq;
      if (active && half == 0) {
        a.P.m[base + q] = -INFINITY;
        a.P.l[base + q] = 0.f;
      }
      t += nv;
      continue;
    }
    if (first_seg) deliver_q(x);   // later segments' queries were delivered while the segment before them ended
    first_seg = false;
    if (stamp) ev[0] = att_timer_ns();
    float m_used = -INFINITY, l_sum = 0.f;
    for (int i = 0; i < n; ++i) {
      const int g = gt + i, sb = g & 1;
      const uint32_t par = (uint32_t)(g >> 1) & 1u;
      int ok = 1;
      if (lane == 0) ok = a5_wait(rg, &ab->s_full[sb], par, 7, g) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) return false;
      if (stamp && i == 0) ev[3] = att_timer_ns();
      att_mbar_try(att_smem_u32(&ab->s_full[sb]), par);   // every lane observes the completed phase
      tc_fence_after();
      const uint32_t s_addr = lane_addr + (uint32_t)(sb * 128 + 64 * half);
      const int n_valid = min(kA5Keys, x.L - (x.ti + i) * kA5Keys) - 64 * half;   // this thread's keys >= n_valid are masked
      // Two passes over the thread's 64 scores, 32 at a time (the maximum first, then the probabilities): tensor memory
      // is cheap to read twice, and 64 scores held in registers beside the epilogues' state made the kernel spill.
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
      for (int c0 = 0; c0 < 64; c0 += 32) {
        float sc[32];
        tc_ld32(s_addr + (uint32_t)c0, sc);
#pragma unroll
        for (int j = 0; j < 32; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], (c0 + j < n_valid) ? sc[j] : -INFINITY);
      }
      float m_tile = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      if (!active) m_tile = 0.f;   // a row slot without a query holds whatever its lane computed: keep it from moving the stabiliser
      mx_own[128 * sb] = m_tile;
      if (!pair_sync()) return false;
      m_tile = fmaxf(m_tile, mx_other[128 * sb]);
      // the stabiliser only moves when the maximum outgrows it by more than 8 (p stays below 256)
      float m_new = m_used, f = 1.f;
      if (m_used == -INFINITY) m_new = m_tile;
      else if (m_tile > m_used + 8.f) { m_new = m_tile; f = ex2_approx(m_used - m_new); }
      if (i > 0 && __any_sync(0xffffffffu, f != 1.f)) {
        // rescale this thread's half of its row of both output accumulators: the previous tile's, once its P V has
        // completed (this tile's cannot start before every thread has delivered its P), and, from the segment's third
        // tile on, this tile's own (its last P V completed before the scores just read were computed: same issuer)
        const uint32_t po = (uint32_t)((g - 1) >> 1) & 1u;
        if (lane == 0) ok = a5_wait(rg, &ab->o_done[(g - 1) & 1], po, 8, g) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) return false;
        att_mbar_try(att_smem_u32(&ab->o_done[(g - 1) & 1]), po);
        tc_fence_after();
#pragma unroll 1
        for (int k = 0; k < (i >= 2 ? 2 : 1); ++k) {
          const uint32_t o_addr = lane_addr + (uint32_t)(256 + 128 * ((g - 1 + k) & 1));
#pragma unroll 1
          for (int c0 = 64 * half; c0 < 64 * half + 64; c0 += 32) {
            float o[32];
            tc_ld32(o_addr + c0, o);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] *= f;
            tc_st32f(o_addr + c0, o);
          }
        }
        tc_wait_st();
        l_sum *= f;
      }
      // probabilities as two bf16 terms over the scores: chunk of 32 keys -> [hi 16 columns | lo 16 columns]; hi = p
      // truncated to bf16, lo = the rest rounded to bf16 (16 significant bits in all)
      float ls4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
      for (int c0 = 0; c0 < 64; c0 += 32) {
        float sc[32];
        tc_ld32(s_addr + (uint32_t)c0, sc);
        if (c0 + 32 > n_valid) {   // warp-uniform; only in a sequence's last tile
#pragma unroll
          for (int j = 0; j < 32; ++j) sc[j] = (c0 + j < n_valid) ? sc[j] : -INFINITY;
        }
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          const float p0 = ex2_approx(sc[j] - m_new), p1 = ex2_approx(sc[j + 1] - m_new);   // 0 for masked keys
          ls4[(j >> 1) & 3] += p0 + p1;
          const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
          hi[j >> 1] = __byte_perm(b0, b1, 0x7632);
          const __nv_bfloat162 bl = __floats2bfloat162_rn(p0 - __uint_as_float(b0 & 0xffff0000u), p1 - __uint_as_float(b1 & 0xffff0000u));
          lo[j >> 1] = *reinterpret_cast<const uint32_t*>(&bl);
        }
        tc_st16(s_addr + (uint32_t)c0, hi);
        tc_st16(s_addr + (uint32_t)c0 + 16, lo);
      }
      l_sum += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
      tc_wait_st();
      tc_fence_before();
      att_mbar_arrive(att_smem_u32(&ab->p_full[sb]));
      m_used = m_new;
    }
    if (stamp) ev[1] = att_timer_ns();
    // The next segment's queries, before this one is wound up: every score MMA of this segment has completed (this
    // thread saw the scores of its last tile), so the query area is free, and the issuers start on the next segment's
    // scores while the partial below is read out (its first P V waits for probabilities that this thread delivers only
    // afterwards, so the output accumulators are not touched early).
    for (long long t2 = t + nv; t2 < t_hi;) {
      AttTile x2;
      int n2, nv2;
      run_at(t2, x2, n2, nv2);
      if (n2 > 0) {
        deliver_q(x2);
        break;
      }
      t2 += nv2;
    }
    // the segment's partial: wait for the last P V of either issuer, then (m, l, o) of every real query row
    {
      const int g = gt + n - 1;
      int ok = 1;
      if (lane == 0)
        ok = (a5_wait(rg, &ab->o_done[g & 1], (uint32_t)(g >> 1) & 1u, 9, g) &&
              (n < 2 || a5_wait(rg, &ab->o_done[(g - 1) & 1], (uint32_t)((g - 1) >> 1) & 1u, 9, g))) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) return false;
      att_mbar_try(att_smem_u32(&ab->o_done[g & 1]), (uint32_t)(g >> 1) & 1u);
      if (n >= 2) att_mbar_try(att_smem_u32(&ab->o_done[(g - 1) & 1]), (uint32_t)((g - 1) >> 1) & 1u);
      tc_fence_after();
      mx_own[128 * ((g + 1) & 1)] = l_sum;   // the buffer the last tile did not use
      if (!pair_sync()) return false;
      const float l_tot = l_sum + mx_other[128 * ((g + 1) & 1)];
      const size_t base = (((size_t)slot0 + (size_t)x.b * Hkv + x.h) * kAttMaxSub + 0) * (size_t)nq;
      if (active && half == 0) {
        a.P.m[base + q] = m_used;
        a.P.l[base + q] = l_tot;
      }
#pragma unroll 1
      for (int c0 = 64 * half; c0 < 64 * half + 64; c0 += 32) {
        float o[32];
        tc_ld32(lane_addr + (uint32_t)(256 + 128 * (g & 1)) + c0, o);
        if (n >= 2) {   // the other issuer's accumulator holds the other half of the segment's tiles
          float o2[32];
          tc_ld32(lane_addr + (uint32_t)(256 + 128 * ((g - 1) & 1)) + c0, o2);
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] += o2[j];
        }
        if (active) {
          float4* dst = reinterpret_cast<float4*>(a.P.o + (base + q) * HD + c0);
#pragma unroll
          for (int j = 0; j < 8; ++j) dst[j] = make_float4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
        }
      }
      tc_fence_before();
      if (!pair_sync()) return false;   // the sums have been read before the next segment's first tile reuses the buffer
      if (stamp) ev[2] = att_timer_ns();
    }
    gt += n;
    t += nv;
  }
  return true;
}

}  // namespace sj
