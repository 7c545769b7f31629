// Weight-streaming skinny GEMM on the 5th-generation tensor cores (sm_100a):
//   D[128 features, R rows] (fp32, TMEM) = W_tile[128, K] (bf16, K-major) x A[R, K]^T (bf16, K-major)
// The weight tile is the MMA's M operand (operands swapped: R is 5..288, far below 128), the
// activations are the N operand.  TMA streams 128x64 weight boxes and Rx64 activation boxes into a
// shared-memory ring (128-byte swizzle); one elected thread issues tcgen05.mma; the accumulator
// lives in TMEM (double-buffered when it fits) and is drained by four epilogue warps.
//
// Work split ("stream-K"): work units are (tile, 64-wide K block) pairs in tile-major order; block c
// owns units [c*U/G, (c+1)*U/G).  Every maximal run of units of one tile inside a block's range is
// a segment; its partial sums go to slot (c - first block of that tile) of the partial buffer and
// are added by the consumer kernel in slot order (deterministic, no atomics).
//
// The LM-head variant splits at whole tiles and replaces the partial store by the fused epilogue:
// per (vocabulary tile, row) softmax statistics (max, sum of exp, arg max), the logit of the
// drafted token, and (only when asked) the raw logits.
//
// Weights do not depend on the previous kernel, so their first ring-full of boxes is requested
// BEFORE the programmatic-dependency wait; activations after it.  Every wait is bounded.
#pragma once

#include <cuda.h>

#include "sj_kernels.cuh"

namespace sj {

constexpr int kBK = 64;                       // K elements per pipeline stage (128 bytes of bf16)
constexpr int kWTileBytes = kTileN * kBK * 2; // 16 KiB
constexpr int kTcThreads = 192;               // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr uint32_t kSpinLimit = 1u << 24;     // bounded waits (~ seconds with the back-off below)

struct TcGemmParams {
  int n_tiles, KB, G;
  long long U;          // n_tiles * KB
  int R;                // valid rows
  int lo_off;           // > 0: activations come as hi/lo bf16 planes; the lo plane's accumulator
                        // columns start at lo_off and are added to the hi columns in the epilogue
  int NB, nblk;         // the accumulator holds NB blocks of nblk rows (nblk % 16 == 0, <= 256)
  int a_blocks;         // activation blocks of nblk rows per stage: NB, or 2 * NB when the hi and the lo plane
                        // are accumulated into the SAME columns (block i adds into accumulator block i % NB)
  int plane_rows;       // row of the lo plane's first block in the activation matrix (used when a_blocks > NB)
  int N_total;          // output features (all segments)
  int seg_tile_end[3];  // exclusive prefix of tiles per weight segment
  int stages;
  int a_stage_bytes;    // a_blocks*nblk*128 rounded up to 1024
  uint32_t tmem_cols;   // power of two >= 32
  int acc_bufs;         // 1 or 2
  int acc_stride;       // columns per accumulator buffer
  float* P;             // partial buffer (split mode)
  size_t slot_stride;
  const int2* tile_slots;
  int lm_mode;          // 1: fused LM-head epilogue, split at whole tiles; 2: same split, raw logits stored to w.logits
                        // [R, V] and nothing else (the second pass over one row per sequence in sampling mode)
  int* status;
};

// ---- PTX wrappers ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking look at a barrier phase (try_wait may suspend the thread for a while before it answers: right
// for a dedicated waiter, wrong for a thread that polls several barriers in turn).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` polls or when another thread of the block gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          uint32_t limit = kSpinLimit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 64) {
      if (*abort_flag) return false;
      __nanosleep(i > 4096 ? 256 : 32);
    }
  }
  *abort_flag = 1;
  atomicCAS(status, DEV_OK, DEV_TIMEOUT);
  return false;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same MMA with the A operand (128 rows x 16 bf16 = 8 columns of 32 bits per row) in tensor memory.
__device__ __forceinline__ void tc_mma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Copy 128 rows x 32 bytes of a shared-memory tile (described like an MMA operand; one 16-element K step of a
// 128-byte-swizzled bf16 tile) into tensor memory: row i to lane i, 8 columns from `taddr`.
__device__ __forceinline__ void tc_cp_128x256b(uint32_t taddr, uint64_t s_desc) {
  asm volatile("tcgen05.cp.cta_group::1.128x256b [%0], %1;" ::"r"(taddr), "l"(s_desc) : "memory");
}
__device__ __forceinline__ void tc_ld8(uint32_t taddr, float* v) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, rows 128 B apart, 8-row groups
// 1024 B apart (stride byte offset), descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);        // start address, 16-byte units
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset
  d |= (uint64_t)1 << 46;                         // version
  d |= (uint64_t)2 << 61;                         // SWIZZLE_128B
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

struct TcSmemCtl {
  uint64_t full[16];
  uint64_t empty[16];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  int tgt_tok[kMaxRows];
  float tgt_pre[kMaxRows];   // top-k test: the drafted tokens' logits, known before the head runs
  RowStat wstat[4][16];  // per epilogue warp, one group of 16 rows at a time
};

__global__ void __launch_bounds__(kTcThreads, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW0,
          const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmW2, TcGemmParams p,
          const StepArgs* __restrict__ args, Work w, int V) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int stage_bytes = kWTileBytes + p.a_stage_bytes;
  TcSmemCtl* ctl = reinterpret_cast<TcSmemCtl*>(smem + (size_t)p.stages * stage_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &ctl->abort_flag;

  // this block's unit range
  const int c = blockIdx.x;
  long long u_lo, u_hi;
  if (p.lm_mode) {
    u_lo = ((long long)c * p.n_tiles / p.G) * p.KB;
    u_hi = ((long long)(c + 1) * p.n_tiles / p.G) * p.KB;
  } else {
    u_lo = (long long)c * p.U / p.G;
    u_hi = (long long)(c + 1) * p.U / p.G;
  }
  const int n_units = (int)(u_hi - u_lo);

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(smem_u32(&ctl->full[i]), 1);
      mbar_init(smem_u32(&ctl->empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&ctl->tmem_full[i]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[i]), 128);
    }
    ctl->abort_flag = 0;
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
  pdl_launch();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      const uint64_t pol_w = l2_policy_evict_first(), pol_a = l2_policy_evict_last();
      const uint32_t tx_bytes = kWTileBytes + (uint32_t)p.a_blocks * p.nblk * 128;
      auto w_load = [&](int it) {
        long long u = u_lo + it;
        int tile = (int)(u / p.KB), kb = (int)(u % p.KB);
        int s = it % p.stages;
        const CUtensorMap* tm = &tmW0;
        int t0 = 0;
        if (tile >= p.seg_tile_end[0]) { tm = &tmW1; t0 = p.seg_tile_end[0]; }
        if (tile >= p.seg_tile_end[1]) { tm = &tmW2; t0 = p.seg_tile_end[1]; }
        uint32_t bar = smem_u32(&ctl->full[s]);
        mbar_expect_tx(bar, tx_bytes);
        tma_load_2d(smem_u32(smem + (size_t)s * stage_bytes), tm, bar, kb * kBK, (tile - t0) * kTileN, pol_w);
      };
      auto a_load = [&](int it) {
        long long u = u_lo + it;
        int kb = (int)(u % p.KB);
        int s = it % p.stages;
        uint32_t bar = smem_u32(&ctl->full[s]);
        for (int nb = 0; nb < p.a_blocks; ++nb)
          tma_load_2d(smem_u32(smem + (size_t)s * stage_bytes + kWTileBytes + (size_t)nb * p.nblk * 128), &tmA, bar,
                      kb * kBK, (nb / p.NB) * p.plane_rows + (nb % p.NB) * p.nblk, pol_a);
      };
      const int pre = min(p.stages, n_units);
      for (int it = 0; it < pre; ++it) w_load(it);   // weights never depend on the previous kernel
      pdl_wait();
      for (int it = 0; it < pre; ++it) a_load(it);
      for (int it = pre; it < n_units; ++it) {
        int s = it % p.stages, round = it / p.stages;
        if (!mbar_wait(smem_u32(&ctl->empty[s]), (round - 1) & 1, abort_flag, p.status)) break;
        w_load(it);
        a_load(it);
      }
    } else {
      pdl_wait();
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    pdl_wait();
    if (lane == 0 && n_units > 0) {
      const uint32_t idesc = instr_desc_bf16(p.nblk);
      int it = 0, seg = 0;
      long long u = u_lo;
      bool alive = true;
      while (u < u_hi && alive) {
        int kb0 = (int)(u % p.KB);
        int len = (int)min((long long)(p.KB - kb0), u_hi - u);
        int acc = seg % p.acc_bufs, use = seg / p.acc_bufs;
        if (use > 0 && !mbar_wait(smem_u32(&ctl->tmem_empty[acc]), (use - 1) & 1, abort_flag, p.status)) break;
        tc_fence_after();
        for (int i = 0; i < len; ++i, ++it) {
          int s = it % p.stages;
          if (!mbar_wait(smem_u32(&ctl->full[s]), (it / p.stages) & 1, abort_flag, p.status)) { alive = false; break; }
          tc_fence_after();
          uint32_t wa = smem_u32(smem + (size_t)s * stage_bytes);
          uint64_t dw = smem_desc_sw128(wa);
          for (int nb = 0; nb < p.a_blocks; ++nb) {
            uint64_t da = smem_desc_sw128(wa + kWTileBytes + nb * p.nblk * 128);
            uint32_t dcol = tmem_base + acc * p.acc_stride + (nb % p.NB) * p.nblk;
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)
              tc_mma_bf16(dcol, dw + 2 * k, da + 2 * k, idesc, (i > 0 || k > 0 || nb >= p.NB) ? 1u : 0u);
          }
          tc_commit(smem_u32(&ctl->empty[s]));  // frees the ring slot once these MMAs have read it
        }
        if (!alive) break;
        tc_commit(smem_u32(&ctl->tmem_full[acc]));
        u += len;
        ++seg;
      }
    }
  } else {
    // ------------------------------ epilogue (4 warps) ------------------------------
    pdl_wait();
    const int quarter = warp & 3;  // TMEM lanes 32*quarter .. +31 belong to this warp
    const int et = threadIdx.x - 64;
    if (p.lm_mode == 1) {
      const int rows = args->gamma + 1;
      for (int r = et; r < p.R; r += 128) {
        int b = r / rows, j = r % rows;
        ctl->tgt_tok[r] = (j < args->gamma) ? args->draft_ids[b * args->gamma + j] : -1;
        ctl->tgt_pre[r] = args->top_k >= 2 ? w.tgt_pre[r] : 0.f;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    const float invT = p.lm_mode ? args->inv_temperature : 1.f;
    const bool topk = p.lm_mode == 1 && args->top_k >= 2;
    float* dbg_logits = p.lm_mode ? args->dbg_logits : nullptr;
    int seg = 0;
    long long u = u_lo;
    while (u < u_hi) {
      int tile = (int)(u / p.KB), kb0 = (int)(u % p.KB);
      int len = (int)min((long long)(p.KB - kb0), u_hi - u);
      int acc = seg % p.acc_bufs, use = seg / p.acc_bufs;
      if (!mbar_wait(smem_u32(&ctl->tmem_full[acc]), use & 1, abort_flag, p.status)) break;
      tc_fence_after();
      const int n = tile * kTileN + quarter * 32 + lane;  // output feature / vocabulary id
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * p.acc_stride;
      if (!p.lm_mode) {
        float* dst = p.P + (size_t)(c - p.tile_slots[tile].x) * p.slot_stride + n;
        for (int c0 = 0; c0 < p.R; c0 += 16) {
          float v[16];
          tc_ld16(taddr + c0, v);
          if (p.lo_off) {
            float lo[16];
            tc_ld16(taddr + p.lo_off + c0, lo);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] += lo[i];
          }
          if (n < p.N_total) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
              if (c0 + i < p.R) dst[(size_t)(c0 + i) * p.N_total] = v[i];
          }
        }
      } else {
        for (int c0 = 0; c0 < p.R; c0 += 16) {
          float v[16];
          tc_ld16(taddr + c0, v);
          if (p.lo_off) {
            float lo[16];
            tc_ld16(taddr + p.lo_off + c0, lo);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] += lo[i];
          }
          if (p.lm_mode == 2) {
            if (n < V) {
#pragma unroll
              for (int i = 0; i < 16; ++i)
                if (c0 + i < p.R) w.logits[(size_t)(c0 + i) * V + n] = v[i];
            }
            continue;
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int r = c0 + i;
            float z = -INFINITY;
            if (r < p.R && n < V) {
              if (w.logits) w.logits[(size_t)r * V + n] = v[i];
              if (dbg_logits) dbg_logits[(size_t)r * V + n] = v[i];
              z = v[i] * invT;
              if (n == ctl->tgt_tok[r]) w.tgt_logit[r] = z;
            }
            float m = z;
            int arg = n;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              float om = __shfl_xor_sync(0xffffffffu, m, o);
              int oa = __shfl_xor_sync(0xffffffffu, arg, o);
              if (om > m || (om == m && oa < arg)) { m = om; arg = oa; }
            }
            float e = (z == -INFINITY) ? 0.f : expf(z - m);
            e = warp_sum(e);
            int before = 0;
            if (topk) {   // block-uniform
              const int tg = r < p.R ? ctl->tgt_tok[r] : -1;
              const float zd = r < p.R ? ctl->tgt_pre[r] : 0.f;
              const bool bf = r < p.R && n < V && tg >= 0 && n != tg && (v[i] > zd || (v[i] == zd && n < tg));
              before = __popc(__ballot_sync(0xffffffffu, bf));
            }
            if (lane == 0) {
              RowStat st; st.m = m; st.s = e; st.arg = arg; st.pad = before;
              ctl->wstat[quarter][i] = st;
            }
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (et < 16 && c0 + et < p.R) {
            RowStat a = ctl->wstat[0][et];
            a = stat_merge(a, ctl->wstat[1][et]);
            a = stat_merge(a, ctl->wstat[2][et]);
            a = stat_merge(a, ctl->wstat[3][et]);
            w.stats[(size_t)tile * p.R + c0 + et] = a;
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
      }
      tc_fence_before();
      mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
      u += len;
      ++seg;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    if (*abort_flag) __nanosleep(20000);  // let copies still in flight land before the block retires
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

}  // namespace sj
