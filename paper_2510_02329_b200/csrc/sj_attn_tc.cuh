// Tensor-core attention of the verification step (bf16 models): causal grouped-query attention of the
// gamma+1 block rows of every sequence over the paged cache, split along the keys over all SMs.
//
// Work decomposition.  The cached keys [0, L_b) of sequence b are cut into ring tiles of KPS keys
// (one tile = 16 KiB: KPS keys of K and of V of one KV head; KPS = 32 for head_dim 128, 64 for head_dim
// 64).  Tiles are ordered (sequence, KV head, tile) and block c owns tiles [c*T/G, (c+1)*T/G); every
// maximal run of tiles of one (sequence, KV head) inside a block's range is a segment.  The block's own
// gamma+1 new rows (positions L_b ..) are a separate "tail" segment per (sequence, KV head), read with
// plain loads from the fp16 copy of those rows that the QKV epilogue writes beside the bf16 pages.  A segment's result is an unnormalised partial (running max m in the
// log2 domain, sum l, output o) per query row; a combine pass merges the partials of a (sequence, KV
// head) in a fixed order (deterministic).
//
// Per segment the query rows of the KV head's group (q = g*(gamma+1) + j, g = head inside the group)
// form the M dimension of mma.sync.m16n8k16 tiles: warp (mi, ks) of a block owns m-tile mi (16 query
// rows) and the ks-th share of the keys of every ring tile, with its own online-softmax state, so
// warps never exchange data; each writes its own sub-partial.
//
// Ring tiles arrive by TMA (tensor map over the page pool, box = 16 slots x 64 dims, 128-byte swizzle)
// into shared memory; K fragments are read with ldmatrix, V fragments with ldmatrix.trans.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "sj_kernels.cuh"

namespace sj {

constexpr int kAttStageBytes = 16384;     // one ring tile: K part then V part, 8 KiB each
constexpr int kAttMaxWarps = 8;           // consumer warps per block
constexpr int kAttMaxSub = 4;             // sub-partials per segment (key shares)
constexpr uint32_t kAttSpin = 1u << 22;

__device__ __forceinline__ uint32_t att_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// The attention MMAs run in fp16 (fp32 accumulate): queries and probabilities are rounded to 11 significant
// bits instead of bf16's 8 (with random values the relative error of an attention output equals the relative
// rounding error of the probabilities, and bf16 probabilities cost 3e-3 of hidden-state accuracy per layer),
// and the cache's bf16 K/V fragments are converted on the fly, exactly for magnitudes in [6e-5, 65504].
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 t = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
// what packing (lo, hi) into fp16 dropped: (lo - fp16(lo), hi - fp16(hi)) as packed fp16; `packed` = pack_f16(lo, hi)
__device__ __forceinline__ uint32_t pack_f16_rest(float lo, float hi, uint32_t packed) {
  const float2 r = __half22float2(*reinterpret_cast<const __half2*>(&packed));
  return pack_f16(lo - r.x, hi - r.y);
}
// two packed bf16 -> two packed fp16
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t x) {
  return pack_f16(__uint_as_float(x << 16), __uint_as_float(x & 0xffff0000u));
}
__device__ __forceinline__ uint32_t ldcg_u32(const void* p) { return __ldcg(reinterpret_cast<const unsigned int*>(p)); }
__device__ __forceinline__ uint32_t ldcg_u16(const void* p) { return (uint32_t)__ldcg(reinterpret_cast<const unsigned short*>(p)); }

// Geometry shared by the attention pass, the combine pass and the host.
struct AttGeom {
  int HD, KPS, MT, KS, KW, nq, rows, group;
};
__host__ __device__ __forceinline__ AttGeom att_geom(int hd, int group, int rows) {
  AttGeom g;
  g.HD = hd;
  g.KPS = kAttStageBytes / (4 * hd);          // keys per ring tile
  g.rows = rows;
  g.group = group;
  g.nq = group * rows;
  g.MT = (g.nq + 15) / 16;
  int ks = g.KPS / 16, cap = kAttMaxWarps / g.MT;
  if (ks > cap) ks = cap;
  if (ks > kAttMaxSub) ks = kAttMaxSub;
  if (ks < 1) ks = 1;
  g.KS = ks == 3 ? 2 : ks;                    // power of two
  g.KW = g.KPS / g.KS;                        // keys per warp per tile
  return g;
}

// Which block owns ring tile t when T tiles are dealt to G blocks as [c*T/G, (c+1)*T/G).
__device__ __forceinline__ int att_owner(long long t, long long T, int G) {
  if (T < (1 << 22) && G < 512) {   // 32-bit arithmetic (64-bit division is slow): t*G and (c+1)*T stay below 2^31
    const unsigned tt = (unsigned)t, TT = (unsigned)T, GG = (unsigned)G;
    unsigned c = tt * GG / TT;
    while ((c + 1) * TT / GG <= tt) ++c;
    return (int)c;
  }
  int c = (int)(t * G / T);
  while ((long long)(c + 1) * T / G <= t) ++c;
  return c;
}

// Partial storage: slot s, sub-partial ks, query row q.
struct AttPartials {
  float* m;   // [slots][kAttMaxSub][nq]
  float* l;
  float* o;   // [slots][kAttMaxSub][nq][hd]
};

// One warp's share of one segment.
template <int HD, int NT>
struct AttWarp {
  uint32_t qa[HD / 16][4];
  float o[HD / 8][4];
  float m0, m1, l0, l1;

  __device__ __forceinline__ void reset() {
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    m0 = m1 = -INFINITY;
    l0 = l1 = 0.f;
  }

  // A fragments of this warp's 16 query rows.  Qb: [nq][HD] fp16 of one (sequence, KV head), already
  // scaled by log2(e)/sqrt(HD).  Rows >= nq repeat row nq-1 (their results are never stored): the loads are
  // unpredicated, so that all of them are in flight together.
  __device__ __forceinline__ void load_q(const __half* __restrict__ Qb, int row0, int nq, int lane) {
    const int r0 = min(row0 + (lane >> 2), nq - 1), r1 = min(row0 + (lane >> 2) + 8, nq - 1), c = (lane & 3) * 2;
#pragma unroll
    for (int k = 0; k < HD / 16; ++k) {
      qa[k][0] = ldcg_u32(Qb + (size_t)r0 * HD + k * 16 + c);
      qa[k][1] = ldcg_u32(Qb + (size_t)r1 * HD + k * 16 + c);
      qa[k][2] = ldcg_u32(Qb + (size_t)r0 * HD + k * 16 + c + 8);
      qa[k][3] = ldcg_u32(Qb + (size_t)r1 * HD + k * 16 + c + 8);
    }
  }

  // Online-softmax update from the score fragments s (log2 domain; masked entries are -inf), returning
  // the probabilities in s.
  __device__ __forceinline__ void softmax_update(float (*s)[4]) {
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
      mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float n0 = fmaxf(m0, mx0), n1 = fmaxf(m1, mx1);
    const float a0 = (m0 == -INFINITY) ? 0.f : exp2f(m0 - n0);
    const float a1 = (m1 == -INFINITY) ? 0.f : exp2f(m1 - n1);
    m0 = n0;
    m1 = n1;
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      s[n][0] = (s[n][0] == -INFINITY) ? 0.f : exp2f(s[n][0] - n0);
      s[n][1] = (s[n][1] == -INFINITY) ? 0.f : exp2f(s[n][1] - n0);
      s[n][2] = (s[n][2] == -INFINITY) ? 0.f : exp2f(s[n][2] - n1);
      s[n][3] = (s[n][3] == -INFINITY) ? 0.f : exp2f(s[n][3] - n1);
      s0 += s[n][0] + s[n][1];
      s1 += s[n][2] + s[n][3];
    }
    l0 = l0 * a0 + s0;
    l1 = l1 * a1 + s1;
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      o[i][0] *= a0; o[i][1] *= a0;
      o[i][2] *= a1; o[i][3] *= a1;
    }
  }

  // One ring tile in shared memory.  `stage`: shared address of the tile (1024-byte aligned): K boxes
  // [page][half] of 2 KiB (16 slots x 64 dims, 128-byte swizzle) then, 8 KiB in, the V boxes.
  // kw0: first key of this warp's share inside the tile; key_abs0: absolute index of that key; L: keys
  // >= L are masked.
  // qlo != nullptr: two-term mode.  The scores also take q_lo . k (the part of the query that its fp16 rounding
  // dropped; qa is overwritten with those fragments and reloaded from qhi afterwards: no second fragment
  // array has to stay in registers), and the probabilities enter the second MMA as p_hi + p_lo.
  // (TWO is a template parameter so that the one-term code, which nearly every layer runs, is compiled exactly as
  // it would be without the two-term mode.)
  template <bool TWO>
  __device__ __forceinline__ void tile(uint32_t stage, int kw0, int key_abs0, int L, int lane, const __half* qhi = nullptr,
                                       const __half* qlo = nullptr, int row0 = 0, int nq = 0) {
    constexpr int HB = HD / 64;
    const int lr = lane & 7, mid = lane >> 3;
    // All K fragments of this warp's keys first (the ldmatrix results are not needed until the MMA chain
    // reaches them; issued one by one in front of their MMA they would serialise the chain), then the V
    // fragments, whose latency hides behind the score MMAs and the softmax arithmetic.
    uint32_t kf[HD / 32][NT][4];
#pragma unroll
    for (int kp = 0; kp < HD / 32; ++kp) {
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        const int kk = kw0 + n * 8 + lr, page = kk >> 4, r = kk & 15;
        const int d = kp * 32 + mid * 8, half = d >> 6, c = (d & 63) >> 3;
        const uint32_t addr = stage + (uint32_t)((page * HB + half) * 2048 + r * 128 + ((c ^ (r & 7)) << 4));
        ldsm_x4(addr, kf[kp][n][0], kf[kp][n][1], kf[kp][n][2], kf[kp][n][3]);
#pragma unroll
        for (int e = 0; e < 4; ++e) kf[kp][n][e] = bf16x2_to_f16x2(kf[kp][n][e]);
      }
    }
    uint32_t vf[NT / 2][HD / 16][4];
#pragma unroll
    for (int kk2 = 0; kk2 < NT / 2; ++kk2) {
#pragma unroll
      for (int dp = 0; dp < HD / 16; ++dp) {
        const int kk = kw0 + kk2 * 16 + (mid & 1) * 8 + lr, page = kk >> 4, r = kk & 15;
        const int d = (dp * 2 + (mid >> 1)) * 8, half = d >> 6, c = (d & 63) >> 3;
        const uint32_t addr =
            stage + 8192u + (uint32_t)((page * HB + half) * 2048 + r * 128 + ((c ^ (r & 7)) << 4));
        ldsm_x4_t(addr, vf[kk2][dp][0], vf[kk2][dp][1], vf[kk2][dp][2], vf[kk2][dp][3]);
#pragma unroll
        for (int e = 0; e < 4; ++e) vf[kk2][dp][e] = bf16x2_to_f16x2(vf[kk2][dp][e]);
      }
    }
    float s[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
    for (int kp = 0; kp < HD / 32; ++kp) {
#pragma unroll
      for (int n = 0; n < NT; ++n) {   // the NT chains are independent: interleaved, they overlap each other's latency
        mma_16816(s[n], qa[2 * kp], kf[kp][n][0], kf[kp][n][1]);
        mma_16816(s[n], qa[2 * kp + 1], kf[kp][n][2], kf[kp][n][3]);
      }
    }
    if constexpr (TWO) {
      load_q(qlo, row0, nq, lane);
#pragma unroll
      for (int kp = 0; kp < HD / 32; ++kp) {
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          mma_16816(s[n], qa[2 * kp], kf[kp][n][0], kf[kp][n][1]);
          mma_16816(s[n], qa[2 * kp + 1], kf[kp][n][2], kf[kp][n][3]);
        }
      }
      load_q(qhi, row0, nq, lane);
    }
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      const int k = key_abs0 + n * 8 + (lane & 3) * 2;
      if (k >= L) { s[n][0] = -INFINITY; s[n][2] = -INFINITY; }
      if (k + 1 >= L) { s[n][1] = -INFINITY; s[n][3] = -INFINITY; }
    }
    softmax_update(s);
#pragma unroll
    for (int kk2 = 0; kk2 < NT / 2; ++kk2) {
      uint32_t pa[4];
      pa[0] = pack_f16(s[2 * kk2][0], s[2 * kk2][1]);
      pa[1] = pack_f16(s[2 * kk2][2], s[2 * kk2][3]);
      pa[2] = pack_f16(s[2 * kk2 + 1][0], s[2 * kk2 + 1][1]);
      pa[3] = pack_f16(s[2 * kk2 + 1][2], s[2 * kk2 + 1][3]);
#pragma unroll
      for (int dp = 0; dp < HD / 16; ++dp) {
        mma_16816(o[2 * dp], pa, vf[kk2][dp][0], vf[kk2][dp][1]);
        mma_16816(o[2 * dp + 1], pa, vf[kk2][dp][2], vf[kk2][dp][3]);
      }
      if constexpr (TWO) {
        uint32_t pl[4];
        pl[0] = pack_f16_rest(s[2 * kk2][0], s[2 * kk2][1], pa[0]);
        pl[1] = pack_f16_rest(s[2 * kk2][2], s[2 * kk2][3], pa[1]);
        pl[2] = pack_f16_rest(s[2 * kk2 + 1][0], s[2 * kk2 + 1][1], pa[2]);
        pl[3] = pack_f16_rest(s[2 * kk2 + 1][2], s[2 * kk2 + 1][3], pa[3]);
#pragma unroll
        for (int dp = 0; dp < HD / 16; ++dp) {
          mma_16816(o[2 * dp], pl, vf[kk2][dp][0], vf[kk2][dp][1]);
          mma_16816(o[2 * dp + 1], pl, vf[kk2][dp][2], vf[kk2][dp][3]);
        }
      }
    }
  }

  // The block's own rows: keys kq = 0..rows-1 at positions L + kq, read with plain loads from the fp16
  // copy written earlier in this step (the pages hold the same rows rounded to bf16 for later steps;
  // reading the copy keeps 11 significant bits of the rows that weigh most when the cache is short).
  // Query row q = g*rows + j sees kq <= j.  krow(kq) / vrow(kq) return the fp16 row pointers [HD].
  template <bool TWO, typename KFn, typename VFn>
  __device__ __forceinline__ void tail(KFn krow, VFn vrow, int rows, int row0, int nq, int lane, const __half* qhi = nullptr,
                                       const __half* qlo = nullptr) {
    const int q0 = row0 + (lane >> 2), q1 = q0 + 8;
    const int j0 = q0 % rows, j1 = q1 % rows;
    for (int kbase = 0; kbase < rows; kbase += NT * 8) {
      float s[NT][4];
#pragma unroll
      for (int n = 0; n < NT; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
      for (int pass = 0; pass < (TWO ? 2 : 1); ++pass) {   // two-term mode: q_hi . k, then q_lo . k (see tile())
        if (pass == 1) load_q(qlo, row0, nq, lane);
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          const int key = kbase + n * 8 + (lane >> 2);
          if (kbase + n * 8 < rows) {   // warp-uniform
            const __half* kr = key < rows ? krow(key) : nullptr;
#pragma unroll
            for (int k = 0; k < HD / 16; ++k) {
              uint32_t b0 = kr ? ldcg_u32(kr + k * 16 + (lane & 3) * 2) : 0u;
              uint32_t b1 = kr ? ldcg_u32(kr + k * 16 + (lane & 3) * 2 + 8) : 0u;
              mma_16816(s[n], qa[k], b0, b1);
            }
          }
        }
        if (pass == 1) load_q(qhi, row0, nq, lane);
      }
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        const int k = kbase + n * 8 + (lane & 3) * 2;
        if (k > j0 || k >= rows || q0 >= nq) s[n][0] = -INFINITY;
        if (k + 1 > j0 || k + 1 >= rows || q0 >= nq) s[n][1] = -INFINITY;
        if (k > j1 || k >= rows || q1 >= nq) s[n][2] = -INFINITY;
        if (k + 1 > j1 || k + 1 >= rows || q1 >= nq) s[n][3] = -INFINITY;
      }
      softmax_update(s);
#pragma unroll
      for (int kk2 = 0; kk2 < NT / 2; ++kk2) {
        if (kbase + kk2 * 16 >= rows) continue;   // warp-uniform
        uint32_t pa[4];
        pa[0] = pack_f16(s[2 * kk2][0], s[2 * kk2][1]);
        pa[1] = pack_f16(s[2 * kk2][2], s[2 * kk2][3]);
        pa[2] = pack_f16(s[2 * kk2 + 1][0], s[2 * kk2 + 1][1]);
        pa[3] = pack_f16(s[2 * kk2 + 1][2], s[2 * kk2 + 1][3]);
        uint32_t pl[4] = {0u, 0u, 0u, 0u};
        if constexpr (TWO) {
          pl[0] = pack_f16_rest(s[2 * kk2][0], s[2 * kk2][1], pa[0]);
          pl[1] = pack_f16_rest(s[2 * kk2][2], s[2 * kk2][3], pa[1]);
          pl[2] = pack_f16_rest(s[2 * kk2 + 1][0], s[2 * kk2 + 1][1], pa[2]);
          pl[3] = pack_f16_rest(s[2 * kk2 + 1][2], s[2 * kk2 + 1][3], pa[3]);
        }
        const int ka = kbase + kk2 * 16 + (lane & 3) * 2;   // keys ka, ka+1 (b0) and ka+8, ka+9 (b1)
        const __half* v00 = ka < rows ? vrow(ka) : nullptr;
        const __half* v01 = ka + 1 < rows ? vrow(ka + 1) : nullptr;
        const __half* v10 = ka + 8 < rows ? vrow(ka + 8) : nullptr;
        const __half* v11 = ka + 9 < rows ? vrow(ka + 9) : nullptr;
#pragma unroll
        for (int dn = 0; dn < HD / 8; ++dn) {
          const int d = dn * 8 + (lane >> 2);
          uint32_t b0 = (v00 ? ldcg_u16(v00 + d) : 0u) | ((v01 ? ldcg_u16(v01 + d) : 0u) << 16);
          uint32_t b1 = (v10 ? ldcg_u16(v10 + d) : 0u) | ((v11 ? ldcg_u16(v11 + d) : 0u) << 16);
          mma_16816(o[dn], pa, b0, b1);
          if constexpr (TWO) mma_16816(o[dn], pl, b0, b1);
        }
      }
    }
  }

  // Write this warp's sub-partial.
  __device__ __forceinline__ void store(const AttPartials& P, size_t slot, int sub, int row0, int nq, int lane) {
    float s0 = l0, s1 = l1;
    s0 += __shfl_xor_sync(0xffffffffu, s0, 1);
    s0 += __shfl_xor_sync(0xffffffffu, s0, 2);
    s1 += __shfl_xor_sync(0xffffffffu, s1, 1);
    s1 += __shfl_xor_sync(0xffffffffu, s1, 2);
    const int q0 = row0 + (lane >> 2), q1 = q0 + 8;
    const size_t base = (slot * kAttMaxSub + sub) * (size_t)nq;
    if ((lane & 3) == 0) {
      if (q0 < nq) { P.m[base + q0] = m0; P.l[base + q0] = s0; }
      if (q1 < nq) { P.m[base + q1] = m1; P.l[base + q1] = s1; }
    }
#pragma unroll
    for (int dn = 0; dn < HD / 8; ++dn) {
      const int d = dn * 8 + (lane & 3) * 2;
      if (q0 < nq) *reinterpret_cast<float2*>(P.o + (base + q0) * HD + d) = make_float2(o[dn][0], o[dn][1]);
      if (q1 < nq) *reinterpret_cast<float2*>(P.o + (base + q1) * HD + d) = make_float2(o[dn][2], o[dn][3]);
    }
  }
};

// Ring-tile bookkeeping of one block: sequence lengths, tile prefix, the block's tile range.
struct AttPlan {
  int L[kMaxBatch];          // cached keys per sequence
  int pre[kMaxBatch + 1];    // ring tiles before sequence b (all KV heads)
  long long T;               // total ring tiles
  // Empty tiles counted after the real ones of every (sequence, KV head) with a non-empty cache.  Tiles are dealt to
  // blocks in equal numbers, and a block pays a fixed price for every (sequence, KV head) it touches (queries, the
  // pipeline's start and drain, the partial): counting that price in tiles keeps ragged batches balanced.  Nobody
  // loads or computes an empty tile.
  int pad;
};

// Filled by one full warp (every lane calls it); callers synchronise afterwards.  Lane i takes sequences i, i + 32, ...:
// the cache lengths are loaded side by side (one thread alone would wait for each load in turn, half a microsecond
// apiece at a batch of 32) and the tile counts summed by a warp prefix sum.
__device__ __forceinline__ void att_plan_fill(AttPlan* pl, const int* __restrict__ row_pos, int B, int rows, int Hkv,
                                              int KPS, int lane, int pad = 0) {
  int carry = 0;
  for (int b0 = 0; b0 < B; b0 += 32) {
    const int b = b0 + lane;
    const int L = b < B ? row_pos[b * rows] : 0;
    const int n = (b < B && L > 0) ? Hkv * ((L + KPS - 1) / KPS + pad) : 0;
    int incl = n;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += up;
    }
    if (b < B) {
      pl->L[b] = L;
      pl->pre[b] = carry + incl - n;
    }
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (lane == 0) {
    pl->pre[B] = carry;
    pl->T = carry;
    pl->pad = pad;
  }
}

__device__ __forceinline__ int att_find_seq(const int* pre, int B, int t) {
  int lo = 0, hi = B - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (pre[mid] <= t) lo = mid; else hi = mid - 1;
  }
  return lo;
}

struct AttArgs {
  const __half* Qb;        // [B][Hkv][nq][HD] scaled queries (fp16)
  const __half* Qlo;       // same layout: the part of the queries that Qb's rounding dropped; null = one-term operands
  const __half* KVn;       // [B][Hkv][2][rows][HD] this step's own key / value rows (fp16)
  AttPartials P;
  int n_tail_base;         // slot of tail (b, h): n_tail_base + b*Hkv + h
  int layer;
};

// ---------------------------------------------------------------------------------------------
// ring plumbing shared by the stand-alone kernel and the whole-step kernel
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void att_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void att_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void att_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool att_mbar_try(uint32_t bar, uint32_t parity) {
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
// On a timeout with abort_g set, abort_g[1] records (where | block << 8) and abort_g[2] `extra`, for the
// host's error message.
__device__ __forceinline__ void att_note_timeout(volatile int* abort_g, int where, int extra) {
  if (!abort_g) return;
  if (atomicCAS(const_cast<int*>(abort_g) + 1, 0, where | ((int)blockIdx.x << 8)) == 0) abort_g[2] = extra;
}
// Bounded wait.  abort_flag: the block's flag (shared memory); abort_g: optional device-wide flag that
// other blocks raise; status: device status word.
// (Kept inline on purpose: an out-of-line call makes the caller save its live registers to local memory,
// and with almost all of the SM's memory configured as shared memory a local-memory access costs an L2
// round trip.)
__device__ __forceinline__ bool att_mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                                volatile int* abort_g, int where, int extra, uint32_t limit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (att_mbar_try(bar, parity)) return true;
    if (i > 64) {
      if (*abort_flag) return false;
      if (abort_g && (i & 255) == 0 && *abort_g) { *abort_flag = 1; return false; }
      __nanosleep(i > 4096 ? 128 : 20);
    }
  }
  *abort_flag = 1;
  att_note_timeout(abort_g, where, extra);
  if (abort_g) *abort_g = 1;
  atomicCAS(status, DEV_OK, DEV_TIMEOUT);
  return false;
}
__device__ __forceinline__ bool att_mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                              volatile int* abort_g = nullptr, int where = 0, int extra = 0,
                                              uint32_t limit = kAttSpin) {
  if (att_mbar_try(bar, parity)) return true;
  return att_mbar_wait_slow(bar, parity, abort_flag, status, abort_g, where, extra, limit);
}
__device__ __forceinline__ void att_tma_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

// Issue the TMA loads of ring tile (sequence slot seq, KV head h, tile index ti) into `stage`; the
// caller has already announced kAttStageBytes on `bar`.
// pages: optional shared-memory copy of this tile's page ids (npg entries, already clamped to the
// sequence's last page); without it each id costs the issuing thread a dependent global load.
__device__ __forceinline__ void att_issue_tile(const CUtensorMap* tmKV, const KvView& kv, int layer, int seq, int h, int ti,
                                               int L, int KPS, int HD, uint32_t stage, uint32_t bar,
                                               const int* pages = nullptr) {
  const int HB = HD / 64, npg = KPS / 16;
  const int last_page = (L - 1) / 16;   // L >= 1 for any ring tile
  for (int p = 0; p < npg; ++p) {
    int pi = ti * npg + p;
    if (pi > last_page) pi = last_page;   // keys there are masked; reload a valid page
    const int page = pages ? pages[p] : __ldg(kv.block_table + (size_t)seq * kv.max_pages_per_seq + pi);
    const long long rowK = ((((long long)layer * kv.n_pages + page) * 2 + 0) * kv.n_kv_heads + h) * 16;
    const long long rowV = rowK + (long long)kv.n_kv_heads * 16;
    for (int half = 0; half < HB; ++half) {
      att_tma_2d(stage + (uint32_t)((p * HB + half) * 2048), tmKV, bar, half * 64, (int)rowK);
      att_tma_2d(stage + 8192u + (uint32_t)((p * HB + half) * 2048), tmKV, bar, half * 64, (int)rowV);
    }
  }
}

// Map ring tile t to (sequence, KV head, tile index, tiles of that (sequence, head)).
struct AttTile { int b, h, ti, nt_b, L, nt_real; };   // nt_b counts the plan's empty tiles, nt_real does not
__device__ __forceinline__ AttTile att_locate(const AttPlan& pl, int B, int KPS, int t) {
  AttTile x;
  x.b = att_find_seq(pl.pre, B, t);
  x.L = pl.L[x.b];
  x.nt_real = (x.L + KPS - 1) / KPS;
  x.nt_b = x.nt_real + pl.pad;
  const int rem = t - pl.pre[x.b];
  x.h = rem / x.nt_b;
  x.ti = rem % x.nt_b;
  return x;
}

// The consumer side of a ring shared with other traffic.
struct AttRing {
  uint64_t* full;        // [stages] shared memory barriers
  uint64_t* empty;
  int* cons_cnt;         // [stages] how many consumer warps are done with the stage
  uint8_t* base;         // first stage
  int stage_stride;      // bytes between stages
  int stages;
  volatile int* abort_flag;
  volatile int* abort_g;
  int* status;
  unsigned long long* ev;   // optional: consumer warp 0 stamps [0] queries loaded, [1] last tile done, [2] partial stored
};
__device__ __forceinline__ unsigned long long att_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
  return t;
}

// One m-tile (query rows row0 .. row0+15) of tail segment x = b * Hkv + h: the block's own rows as keys.
template <int HD, int NT>
__device__ __forceinline__ void att_tail_task(AttWarp<HD, NT>& st, const AttGeom& g, const AttArgs& a, int x, int row0, int lane) {
  const int rows = g.rows;
  st.reset();
  const __half* qhi = a.Qb + (size_t)x * g.nq * HD;
  const __half* qlo = a.Qlo ? a.Qlo + (size_t)x * g.nq * HD : nullptr;
  st.load_q(qhi, row0, g.nq, lane);
  const __half* kn = a.KVn + (size_t)x * 2 * rows * HD;
  auto krow = [&](int kq) -> const __half* { return kn + (size_t)kq * HD; };
  auto vrow = [&](int kq) -> const __half* { return kn + (size_t)(rows + kq) * HD; };
  if (qlo) st.template tail<true>(krow, vrow, rows, row0, g.nq, lane, qhi, qlo);   // warp-uniform
  else st.template tail<false>(krow, vrow, rows, row0, g.nq, lane);
  st.store(a.P, (size_t)a.n_tail_base + x, 0, row0, g.nq, lane);
}

// One consumer warp (cw of kAttMaxWarps) of block c of G.  The first n_active = MT*KS warps take all ring
// segments of the block's tile range [t_lo, t_hi) starting at ring position `it`; the others take tail tasks.
template <int HD, int NT>
__device__ __forceinline__ bool att_consume(const AttRing& rg, int& it, const AttPlan& pl, const AttGeom& g,
                                            const StepArgs* __restrict__ args, const KvView& kv, const AttArgs& a, int Hkv,
                                            int c, int G, int cw, int lane) {
  const int B = args->B, n_active = g.MT * g.KS, n_spare = kAttMaxWarps - n_active;
  AttWarp<HD, NT> st;
  if (cw >= n_active) {
    // A consumer warp without a share of the ring tiles takes tail tasks (one m-tile of one tail segment
    // each), dealt over the spare warps of all blocks from the last block down: the tails then run beside
    // the tiles instead of after them.
    for (int q = (G - 1 - c) * n_spare + (cw - n_active); q < B * Hkv * g.MT; q += G * n_spare)
      att_tail_task<HD, NT>(st, g, a, q / g.MT, (q % g.MT) * 16, lane);
    return true;
  }
  const int mi = cw / g.KS, ks = cw % g.KS, row0 = mi * 16;
  const long long T = pl.T;
  const long long t_lo = (long long)c * T / G, t_hi = (long long)(c + 1) * T / G;
  long long t = t_lo;
  while (t < t_hi) {
    const AttTile x = att_locate(pl, B, g.KPS, (int)t);
    const int n = (int)min((long long)(x.nt_b - x.ti), t_hi - t);
    st.reset();
    const __half* qhi = a.Qb + ((size_t)x.b * Hkv + x.h) * g.nq * HD;
    const __half* qlo = a.Qlo ? a.Qlo + ((size_t)x.b * Hkv + x.h) * g.nq * HD : nullptr;
    st.load_q(qhi, row0, g.nq, lane);
    if (rg.ev && cw == 0 && lane == 0) { rg.ev[3] = st.qa[0][0]; rg.ev[0] = att_timer_ns(); }
    for (int i = 0; i < n; ++i, ++it) {
      const int s = it % rg.stages;
      const uint32_t bar = att_smem_u32(&rg.full[s]), par = (uint32_t)(it / rg.stages) & 1u;
      int ok = 1;
      if (lane == 0) ok = att_mbar_wait(bar, par, rg.abort_flag, rg.status, rg.abort_g, 9, it) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) return false;
      att_mbar_try(bar, par);   // every lane observes the completed phase
      __syncwarp();
      if (qlo)   // warp-uniform
        st.template tile<true>(att_smem_u32(rg.base + (size_t)s * rg.stage_stride), ks * g.KW, (x.ti + i) * g.KPS + ks * g.KW, x.L,
                               lane, qhi, qlo, row0, g.nq);
      else
        st.template tile<false>(att_smem_u32(rg.base + (size_t)s * rg.stage_stride), ks * g.KW, (x.ti + i) * g.KPS + ks * g.KW, x.L, lane);
      __syncwarp();
      if (lane == 0) {
        __threadfence_block();
        if (atomicAdd(&rg.cons_cnt[s], 1) == n_active - 1) {
          rg.cons_cnt[s] = 0;
          __threadfence_block();
          att_mbar_arrive(att_smem_u32(&rg.empty[s]));
        }
      }
    }
    if (rg.ev && cw == 0 && lane == 0) rg.ev[1] = att_timer_ns();
    st.store(a.P, (size_t)c + (size_t)x.b * Hkv + x.h, ks, row0, g.nq, lane);
    if (rg.ev && cw == 0 && lane == 0) rg.ev[2] = att_timer_ns();
    t += n;
  }
  // without spare warps: tail segment (b, h) number x goes to block G-1-(x mod G), key share 0 only
  if (n_spare == 0 && ks == 0)
    for (int x = G - 1 - c; x < B * Hkv; x += G) att_tail_task<HD, NT>(st, g, a, x, row0, lane);
  return true;
}

template <int HD>
__device__ __forceinline__ bool att_consume_dispatch(const AttRing& rg, int& it, const AttPlan& pl, const AttGeom& g,
                                                     const StepArgs* __restrict__ args, const KvView& kv, const AttArgs& a,
                                                     int Hkv, int c, int G, int cw, int lane) {
  if (g.KW == 16) return att_consume<HD, 2>(rg, it, pl, g, args, kv, a, Hkv, c, G, cw, lane);
  if (g.KW == 32) return att_consume<HD, 4>(rg, it, pl, g, args, kv, a, Hkv, c, G, cw, lane);
  if constexpr (HD == 64) return att_consume<HD, 8>(rg, it, pl, g, args, kv, a, Hkv, c, G, cw, lane);
  return true;
}

// ---------------------------------------------------------------------------------------------
// stand-alone kernel (used by the multi-kernel step): warp 0 streams the ring, warps 1..8 consume
// ---------------------------------------------------------------------------------------------
constexpr int kAttStages = 8;
constexpr int kAttTcThreads = 32 * (1 + kAttMaxWarps);
constexpr int kAttPageCache = 1024;   // page ids of a block's first tiles kept in shared memory
struct AttSmemCtl {
  uint64_t full[kAttStages];
  uint64_t empty[kAttStages];
  int cons_cnt[kAttStages];
  int abort_flag;
  AttPlan plan;
  int pages[kAttPageCache];
};
// Page ids of the block's ring tiles [t_lo, t_hi), npg per tile, as many as fit; all threads of the caller.
__device__ __forceinline__ void att_fill_pages(int* pages, const AttPlan& pl, const KvView& kv, const StepArgs* args, int B,
                                               int KPS, long long t_lo, long long t_hi, int tid, int nthreads) {
  const int npg = KPS / 16;
  const long long n = min((t_hi - t_lo) * npg, (long long)kAttPageCache);
  for (int i = tid; i < n; i += nthreads) {
    const AttTile x = att_locate(pl, B, KPS, (int)(t_lo + i / npg));
    int pi = x.ti * npg + i % npg;
    const int last_page = (x.L - 1) / 16;
    if (pi > last_page) pi = last_page;
    pages[i] = __ldg(kv.block_table + (size_t)args->seq_ids[x.b] * kv.max_pages_per_seq + pi);
  }
}

template <int HD>
__global__ void __launch_bounds__(kAttTcThreads, 1)
k_attn_tc(const __grid_constant__ CUtensorMap tmKV, const StepArgs* __restrict__ args, KvView kv, Work w, Dims dm,
          AttArgs a) {
  extern __shared__ uint8_t att_smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(att_smem_raw) + 1023) & ~(uintptr_t)1023);
  AttSmemCtl* ctl = reinterpret_cast<AttSmemCtl*>(ring + kAttStages * kAttStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_wait();
  pdl_launch();
  const int B = args->B, rows = args->gamma + 1, Hkv = dm.Hkv;
  const AttGeom g = att_geom(HD, dm.Hq / dm.Hkv, rows);
  if (threadIdx.x == 0) {
    for (int i = 0; i < kAttStages; ++i) {
      att_mbar_init(att_smem_u32(&ctl->full[i]), 1);
      att_mbar_init(att_smem_u32(&ctl->empty[i]), 1);
      ctl->cons_cnt[i] = 0;
    }
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) att_plan_fill(&ctl->plan, w.row_pos, B, rows, Hkv, g.KPS, lane);
  __syncthreads();
  const AttPlan& pl = ctl->plan;
  const int G = gridDim.x, c = blockIdx.x;
  volatile int* abort_flag = &ctl->abort_flag;
  {
    const long long t_lo = (long long)c * pl.T / G, t_hi = (long long)(c + 1) * pl.T / G;
    att_fill_pages(ctl->pages, pl, kv, args, B, g.KPS, t_lo, t_hi, threadIdx.x, blockDim.x);
  }
  __syncthreads();
  if (warp == 0) {
    if (lane == 0) {
      const long long t_lo = (long long)c * pl.T / G, t_hi = (long long)(c + 1) * pl.T / G;
      const int npg = g.KPS / 16;
      int it = 0;
      for (long long t = t_lo; t < t_hi; ++t, ++it) {
        const int s = it % kAttStages, round = it / kAttStages;
        if (round > 0 && !att_mbar_wait(att_smem_u32(&ctl->empty[s]), (round - 1) & 1, abort_flag, w.status)) break;
        const AttTile x = att_locate(pl, B, g.KPS, (int)t);
        const uint32_t bar = att_smem_u32(&ctl->full[s]);
        att_mbar_expect_tx(bar, kAttStageBytes);
        att_issue_tile(&tmKV, kv, a.layer, args->seq_ids[x.b], x.h, x.ti, x.L, g.KPS, HD,
                       att_smem_u32(ring + (size_t)s * kAttStageBytes), bar,
                       (it + 1) * npg <= kAttPageCache ? ctl->pages + it * npg : nullptr);
      }
    }
  } else {
    AttRing rg{ctl->full, ctl->empty, ctl->cons_cnt, ring, kAttStageBytes, kAttStages, abort_flag, nullptr, w.status, nullptr};
    int it = 0;
    att_consume_dispatch<HD>(rg, it, pl, g, args, kv, a, Hkv, c, G, warp - 1, lane);
  }
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) __nanosleep(20000);   // let copies in flight land before the block retires
}

// Merge the partials of one (sequence, KV head, query row): ring segments in block order, their
// sub-partials in key-share order, then the tail.  One warp per item; writes the O-projection input.
// G_att: number of blocks of the attention pass.  Partial buffers are zero-filled at allocation, so the
// slots of blocks without tiles (weight 0) hold finite values.
// 128-bit / 64-bit loads of a lane's share of an output row
template <int DPL> struct AttVec;
template <> struct AttVec<4> {
  typedef float4 type;
  static __device__ __forceinline__ void fma(float* acc, const float4& v, float w) {
    acc[0] += v.x * w; acc[1] += v.y * w; acc[2] += v.z * w; acc[3] += v.w * w;
  }
};
template <> struct AttVec<2> {
  typedef float2 type;
  static __device__ __forceinline__ void fma(float* acc, const float2& v, float w) { acc[0] += v.x * w; acc[1] += v.y * w; }
};

// kAttCombineSplit warps share one item (each a contiguous part of the head dimension): with two, the 2 x 32
// dims a lane holds per sub-partial are one 8-byte load and all sub-partials of a config-3 item (39) are in
// flight at once; with one warp per item they need two dependent batches.
template <int HD> struct AttCombineSplit { static constexpr int value = HD >= 128 ? 2 : 1; };
// OBN: output rows one lane keeps in flight (0: 40 or 24, sized for the 30..40 sub-partials of short tiles; 8 where long
// tiles leave an item a handful of sub-partials: the clamped repeats of the last row would be most of the pass's L2
// traffic)
template <typename T, int HD, int OBN = 0>
__device__ __forceinline__ void att_combine_item(const AttPartials& P, const AttPlan& pl, const AttGeom& g, int G_att,
                                                 int n_tail_base, int Hkv, int item_part, void* ATT, int R, int Hq, int lane,
                                                 unsigned long long* ev = nullptr) {
  constexpr int SPLIT = AttCombineSplit<HD>::value;
  const int item = item_part / SPLIT, part = item_part % SPLIT;
  const int q = item % g.nq, bh = item / g.nq, b = bh / Hkv, h = bh % Hkv;
  const int L = pl.L[b];
  const int nt_b = L > 0 ? (L + g.KPS - 1) / g.KPS + pl.pad : 0;
  int c_first = 0, n_cta = 0;
  if (nt_b > 0) {
    const long long t0 = (long long)pl.pre[b] + (long long)h * nt_b;
    c_first = att_owner(t0, pl.T, G_att);
    n_cta = att_owner(t0 + nt_b - 1, pl.T, G_att) - c_first + 1;
  }
  const int n_sub = n_cta * g.KS + 1;   // the last one is the tail
  // sub-partial k of the ring: block c_first + k / KS, key share k % KS (KS is a power of two); row index in
  // the partial arrays = base + (k / KS) * 4 * nq + (k % KS) * nq
  const int ks_shift = g.KS == 4 ? 2 : (g.KS == 2 ? 1 : 0), ks_mask = g.KS - 1;
  const int base = ((c_first + bh) * kAttMaxSub) * g.nq + q, step_c = kAttMaxSub * g.nq;
  const int tail_idx = ((n_tail_base + bh) * kAttMaxSub) * g.nq + q;
  auto sub_index = [&](int k) -> int {
    return k >= n_sub - 1 ? tail_idx : base + (k >> ks_shift) * step_c + (k & ks_mask) * g.nq;
  };
  const bool all_live = pl.T >= G_att;   // every block of the attention pass owns at least one tile
  auto sub_live = [&](int k) -> bool {
    if (all_live || k == n_sub - 1) return true;
    const int cc = c_first + (k >> ks_shift);
    return (long long)(cc + 1) * pl.T / G_att > (long long)cc * pl.T / G_att;
  };
  constexpr int DPL = HD / 32 / SPLIT;   // dims per lane
  constexpr int OB = OBN > 0 ? OBN : (DPL <= 2 ? 40 : 24);   // output rows whose loads one lane keeps in flight
  constexpr int RS = HD / DPL;             // row stride of the outputs in units of V
  typedef typename AttVec<DPL>::type V;
  const V* Po = reinterpret_cast<const V*>(P.o) + part * 32 + lane;   // row r of the outputs starts at Po + r * RS
  float lsum = 0.f, Mrun = -INFINITY, acc[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
  for (int k0 = 0; k0 < n_sub; k0 += 96) {   // 96 sub-partials at a time (three per lane); one pass in practice
    // Everything this pass reads is requested before anything is used: maxima, sums, and the first OB
    // output rows (their weights are not needed to issue the loads).
    float mk[3], lk[3];
#pragma unroll
    for (int u = 0; u < 3; ++u) {
      const int k = k0 + u * 32 + lane;
      const bool live = k < n_sub && sub_live(k);
      mk[u] = live ? __ldcg(P.m + sub_index(k)) : -INFINITY;
      lk[u] = live ? __ldcg(P.l + sub_index(k)) : 0.f;
    }
    const int kn = min(96, n_sub - k0);
    V ob[OB];
#pragma unroll
    for (int k = 0; k < OB; ++k) ob[k] = __ldcg(Po + (size_t)sub_index(k0 + min(k, kn - 1)) * RS);
    float Mb = fmaxf(fmaxf(mk[0], mk[1]), mk[2]);
    if (ev && lane == 0) ev[0] = att_timer_ns();
    Mb = warp_max(Mb);
    const float Mnew = fmaxf(Mrun, Mb);
    if (Mnew == -INFINITY) continue;   // warp-uniform: nothing live so far
    const float rescale = (Mrun == -INFINITY) ? 0.f : exp2f(Mrun - Mnew);
    lsum *= rescale;
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] *= rescale;
    Mrun = Mnew;
    float wk[3], lpart = 0.f;
#pragma unroll
    for (int u = 0; u < 3; ++u) {
      wk[u] = (mk[u] == -INFINITY) ? 0.f : exp2f(mk[u] - Mnew);
      lpart += lk[u] * wk[u];
    }
    lsum += warp_sum(lpart);
    if (ev && lane == 0) ev[1] = att_timer_ns();
#pragma unroll
    for (int k = 0; k < OB; ++k) {
      const float wgt = k < kn ? __shfl_sync(0xffffffffu, k < 32 ? wk[0] : wk[1], k & 31) : 0.f;
      AttVec<DPL>::fma(acc, ob[k], wgt);
    }
    for (int kb = OB; kb < kn; kb += OB) {   // further output rows, OB at a time, added in order
#pragma unroll
      for (int k = 0; k < OB; ++k) ob[k] = __ldcg(Po + (size_t)sub_index(k0 + min(kb + k, kn - 1)) * RS);
#pragma unroll
      for (int k = 0; k < OB; ++k) {
        const int kk = kb + k;
        const float wsel = kk < 32 ? wk[0] : (kk < 64 ? wk[1] : wk[2]);
        const float wgt = kk < kn ? __shfl_sync(0xffffffffu, wsel, kk & 31) : 0.f;
        AttVec<DPL>::fma(acc, ob[k], wgt);
      }
    }
  }
  if (ev && lane == 0) { ev[3] = (unsigned long long)__float_as_uint(acc[0]); ev[2] = att_timer_ns(); }
  const int gq = q / g.rows, j = q % g.rows, r = b * g.rows + j, head = h * g.group + gq;
  const float inv = 1.0f / lsum;
#pragma unroll
  for (int i = 0; i < DPL; ++i) store_act<T>(ATT, R, Hq * HD, r, head * HD + (part * 32 + lane) * DPL + i, acc[i] * inv);
}

// keys_per_tile > 0: the partials come from a pass that cut the cache into tiles of that many keys (plus tile_pad empty
// ones per (sequence, KV head)) with one sub-partial per block segment (the tcgen05 attention); 0: this file's own
// geometry.
template <int HD, int OBN>
__global__ void k_attn_combine_tc(const StepArgs* __restrict__ args, Work w, Dims dm, AttPartials P, int G_att,
                                  int n_tail_base, int keys_per_tile, int tile_pad) {
  __shared__ AttPlan pl;
  pdl_wait();
  pdl_launch();
  const int B = args->B, rows = args->gamma + 1;
  AttGeom g = att_geom(HD, dm.Hq / dm.Hkv, rows);
  if (keys_per_tile > 0) { g.KPS = keys_per_tile; g.KS = 1; g.KW = keys_per_tile; }
  if (threadIdx.x < 32) att_plan_fill(&pl, w.row_pos, B, rows, dm.Hkv, g.KPS, threadIdx.x, keys_per_tile > 0 ? tile_pad : 0);
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
  const int items = B * dm.Hkv * g.nq * AttCombineSplit<HD>::value;
  for (int item = warp * gridDim.x + blockIdx.x; item < items; item += gridDim.x * wpb)   // spread over blocks first
    att_combine_item<bf16, HD, OBN>(P, pl, g, G_att, n_tail_base, dm.Hkv, item, w.ATT, B * rows, dm.Hq, lane);
}

}  // namespace sj
