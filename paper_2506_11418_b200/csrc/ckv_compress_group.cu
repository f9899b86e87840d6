// Chunked Soft Matching round at chunk 128 and 256 (the paper's default), bf16, head_dim 128, full chunks, the modes
// that merge: every edge, the best m of each chunk, or the flags of a per-head ranking.
//
// Persistent kernel, one CTA per SM.  A group of C / 64 warps owns one shared-memory stage that holds one tensor's tile
// of a chunk (C rows of 256 bytes); several groups per CTA work on different chunks in different phases, so loads,
// matching, merging and stores of different chunks overlap without a CTA-wide barrier.  A chunk goes through its
// group's stage twice: first the K tile (matching, selection, merged keys), then the V tile (the same clusters).
//   fetch     TMA tensor copies, 128-byte swizzle, the tensor map views the cache as (column, parity, token pair,
//             slab): A tokens (1st, 3rd, ...) land in rows 0 .. C/2 - 1 of each 64-column half, B tokens behind them
//   Sec. 5.2  every warp takes 32 A tokens against all B tokens of the chunk, 64 at a time: mma.sync m16n8k16 with
//             ldmatrix fragments, fp32 accumulate; inverse norms from X X^T diagonals; running row argmax of the cosine
//             of Eq. 2 (lowest index on ties)
//   Sec. 5.3  one thread per A token: every edge, rank inside the chunk, or the flag from global memory
//   Eq. 5     every warp produces 32 B rows: C = W X on tensor cores with W [32 x C] = degree of token k in row b if k
//             is b itself or a selected A token matched to b (degrees in exact 8-bit pieces, one pass per piece that
//             occurs), X = the staged tile read column-wise (ldmatrix.trans); blocks of W without an entry are skipped;
//             times 1 / n', rounded to bf16, written over the B row in the tile (stmatrix)
//   store     every edge merged: the B rows are the output, one TMA tensor store per half; otherwise the surviving
//             rows leave in order through a row table with 16-byte stores
// Waits on the mbarrier are bounded: a group that gives up records it in the status word and leaves.
#include <cuda.h>

#include <algorithm>
#include <cstdint>

#include "ckv_common.cuh"
#include "ckv_internal.h"
#include "ckv_ptx.cuh"

namespace ckv {

namespace {

using namespace ptx;

constexpr uint32_t kOneBits = 0x3f80u;  // bf16 1.0

template <int C>
struct GroupCfg {
  static constexpr int kNA = C / 2;             // A tokens = B tokens of a chunk
  static constexpr int kGW = C / 64;            // warps per group: 32 A tokens and 32 B rows each
  static constexpr int kHalf = C * 128;         // one 64-column half of a tile: C rows of 128 bytes, swizzled
  static constexpr int kStage = 2 * kHalf;      // one tensor's tile of a chunk
  static constexpr int kGroups = C == 256 ? 3 : 6;
  static constexpr int kThreads = kGroups * kGW * 32;
  // per group, behind the stages: degrees [C] int (A tokens then B tokens), summed degrees [NA] int, inverse norms of the
  // B keys [NA] float, edge similarities [NA] float, new degrees by output row [C] int, output row table [C] ushort,
  // edge targets [NA] uchar (255 = not merged), selection mask words [4], flags, mbarrier
  static constexpr int oDeg = 0;
  static constexpr int oDsum = oDeg + 4 * C;
  static constexpr int oInvB = oDsum + 4 * kNA;
  static constexpr int oSim = oInvB + 4 * kNA;
  static constexpr int oNewDeg = oSim + 4 * kNA;
  static constexpr int oRowOf = oNewDeg + 4 * C;
  static constexpr int oTgt = oRowOf + 2 * C;
  static constexpr int oMask = oTgt + kNA;
  static constexpr int oFlags = oMask + 16;     // int: largest degree of the chunk
  static constexpr int oBar = oFlags + 8;
  static constexpr int oBar2 = oBar + 8;        // chunk 256: the matching MMAs have completed
  static constexpr int oBlkInv = oBar2 + 8;     // chunk 256: float [4], largest 1 / |b| of every 32 B tokens
  static constexpr int kExtra = (oBlkInv + 16 + 127) / 128 * 128;
  static constexpr int oTmem = kGroups * (kStage + kExtra);  // chunk 256: the CTA's tensor-memory base address
  static constexpr size_t kSmem = (size_t)oTmem + 16;
  // Chunk 256: the 128 x 128 x 128 dot products of a chunk run on the 5th-generation tensor core (tcgen05.mma from the
  // TMA-delivered tile into 128 columns of tensor memory per group); the warps only read the scores back.
  static constexpr bool kUmma = C == 256;
};

// instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 128
__host__ __device__ constexpr uint32_t group_idesc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

// byte address of 16-byte piece c16 (0..15) of row `row` of a swizzled tile whose halves are `half` bytes apart
template <int C>
__device__ __forceinline__ uint32_t g_addr(uint32_t tile, int row, int c16) {
  return tile + (uint32_t)(c16 >> 3) * GroupCfg<C>::kHalf + (uint32_t)row * 128u + (uint32_t)(((c16 & 7) ^ (row & 7)) << 4);
}

// bar.sync among the warps of one group (barrier ids 1 .. kGroups)
__device__ __forceinline__ void group_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// inverse norms of 32 consecutive rows of the tile (row0 .. row0 + 31) from the diagonals of X X^T: lane i gets 1 / |x_i|
// (0 for a zero row)
template <int C>
__device__ __forceinline__ float inv_norms32(uint32_t tile, int row0, int lane) {
  const int g = lane >> 2;
  // B-operand style fragments of two 16-row blocks: matrices (rows 0-7 | columns 0-7, 8-15), (rows 8-15 | ...)
  const int x_row = row0 + (lane & 7) + (lane >> 4) * 8, x_c = (lane >> 3) & 1;
  float nacc[2][2][4];
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    uint32_t f[2][4];
#pragma unroll
    for (int p = 0; p < 2; ++p) ldsm_x4(g_addr<C>(tile, x_row + 16 * p, 2 * kk + x_c), f[p]);
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      if (kk == 0) {
        mma_bf16_first(nacc[p][0], f[p][0], f[p][2], f[p][1], f[p][3], f[p][0], f[p][1]);
        mma_bf16_first(nacc[p][1], f[p][0], f[p][2], f[p][1], f[p][3], f[p][2], f[p][3]);
      } else {
        mma_bf16(nacc[p][0], f[p][0], f[p][2], f[p][1], f[p][3], f[p][0], f[p][1]);
        mma_bf16(nacc[p][1], f[p][0], f[p][2], f[p][1], f[p][3], f[p][2], f[p][3]);
      }
    }
  }
  // the squared norm of row 8 q + g (q = 0..3) sits in lane (g, t = g / 2), register g & 1 (+2 for odd q)
  float mine = 0.f;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int p = q >> 1, hh = q & 1;
    const float ss = (g & 1) ? nacc[p][hh][2 * hh + 1] : nacc[p][hh][2 * hh];
    const float inv = ss > 0.f ? rsqrtf(ss) : 0.f;
    // row 8 q + r lives in lane 4 r + r / 2: lane i = 8 q + r fetches from there
    const float v = __shfl_sync(0xffffffffu, inv, 4 * (lane & 7) + ((lane & 7) >> 1));
    if ((lane >> 3) == q) mine = v;
  }
  return mine;
}

// Sec. 5.2 for 32 A tokens (tile rows a0 .. a0 + 31) against the chunk's NB B tokens (rows NA ...): the row argmax of
// dot * inv_b (the cosine up to the row's own factor 1 / |a|, which cannot change an argmax).  Returns, in lane i, A
// token a0 + i's best B index and that maximum.
template <int C>
__device__ __forceinline__ void match_rows(uint32_t tile, int a0, const float* inv_b, int lane, int& best, float& best_v) {
  constexpr int NA = GroupCfg<C>::kNA;
  const int t = lane & 3;
  const int a_row = a0 + (lane & 7) + ((lane >> 3) & 1) * 8, a_c = lane >> 4;
  const int b_row = NA + (lane & 7) + (lane >> 4) * 8, b_c = (lane >> 3) & 1;
  float row_v[2][2];
  int row_i[2][2];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      row_v[mt][hi] = -INFINITY;
      row_i[mt][hi] = 0x7fffffff;
    }
#pragma unroll 1
  for (int bh = 0; bh < NA / 64; ++bh) {  // 64 B tokens at a time: n tile nt = B indices 64 bh + 8 nt ...
    float acc[2][8][4];
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      uint32_t fa[2][4], fb[4][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) ldsm_x4(g_addr<C>(tile, a_row + 16 * mt, 2 * kk + a_c), fa[mt]);
#pragma unroll
      for (int p = 0; p < 4; ++p) ldsm_x4(g_addr<C>(tile, b_row + 64 * bh + 16 * p, 2 * kk + b_c), fb[p]);
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const uint32_t b0 = fb[nt >> 1][2 * (nt & 1)], b1 = fb[nt >> 1][2 * (nt & 1) + 1];
          if (kk == 0)
            mma_bf16_first(acc[mt][nt], fa[mt][0], fa[mt][1], fa[mt][2], fa[mt][3], b0, b1);
          else
            mma_bf16(acc[mt][nt], fa[mt][0], fa[mt][1], fa[mt][2], fa[mt][3], b0, b1);
        }
    }
    // columns in increasing order within the thread: a strict > keeps the lowest index
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float2 ib = *reinterpret_cast<const float2*>(inv_b + 64 * bh + 8 * nt + 2 * t);
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
          const float s0 = acc[mt][nt][2 * hi] * ib.x + 0.f, s1 = acc[mt][nt][2 * hi + 1] * ib.y + 0.f;  // -0 -> +0
          if (s0 > row_v[mt][hi]) { row_v[mt][hi] = s0; row_i[mt][hi] = 64 * bh + 8 * nt + 2 * t; }
          if (s1 > row_v[mt][hi]) { row_v[mt][hi] = s1; row_i[mt][hi] = 64 * bh + 8 * nt + 2 * t + 1; }
        }
    }
  }
  best = 0;
  best_v = 0.f;
  const int src = 4 * (lane & 7), which = lane >> 3;
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      float bv = row_v[mt][hi];
      int bi = row_i[mt][hi];
#pragma unroll
      for (int o = 1; o <= 2; o <<= 1) {  // the four lanes of a quad hold the same row
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      // lane = A index i takes row i = 16 mt + 8 hi + g from the quad of g = i & 7
      const int vb = __shfl_sync(0xffffffffu, bi, src);
      const float vv = __shfl_sync(0xffffffffu, bv, src);
      if (which == 2 * mt + hi) { best = vb; best_v = vv; }
    }
  best = min(best, NA - 1);  // a row of NaNs has no maximum: stay inside the chunk
}

// The same for chunk 256 from tensor memory: lane i of warp w reads row 32 w + i of the 128 x 128 accumulator (raw dot
// products), 32 columns at a time.  The 32 B tokens around the row's own position come first: with keys that resemble
// their neighbours they set a high mark, and another block of 32 is only examined when its largest dot product times its
// largest 1 / |b| (blk_inv) could reach some lane's mark.  (x <= max and 1/|b| <= blk_inv, all non-negative where it
// matters, and rounding is monotonic: a skipped block holds no better candidate; ties go to the lowest B index.)
__device__ __forceinline__ void match_rows_tmem(uint32_t taddr, int w, const float* inv_b, const float* blk_inv, int& best,
                                                float& best_v) {
  float bv = -INFINITY;
  int bi = 0x7fffffff;
#pragma unroll 1
  for (int k = 0; k < 4; ++k) {
    const int blk = k == 0 ? w : (k <= w ? k - 1 : k);  // own block first, then the others in increasing order
    float v[32];
    tmem_ld32(taddr + (uint32_t)(32 * blk), v);
    if (k > 0) {
      float m0 = fmaxf(v[0], v[1]), m1 = fmaxf(v[2], v[3]);
#pragma unroll
      for (int j = 4; j < 32; j += 4) {
        m0 = fmaxf(m0, fmaxf(v[j], v[j + 1]));
        m1 = fmaxf(m1, fmaxf(v[j + 2], v[j + 3]));
      }
      const float bound = fmaxf(fmaxf(m0, m1), 0.f) * blk_inv[blk];
      if (!__any_sync(0xffffffffu, bound >= bv)) continue;
    }
#pragma unroll
    for (int j = 0; j < 32; j += 4) {
      const float4 ib = *reinterpret_cast<const float4*>(inv_b + 32 * blk + j);
      const float ibs[4] = {ib.x, ib.y, ib.z, ib.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float sc = v[j + e] * ibs[e] + 0.f;  // -0 -> +0
        const int idx = 32 * blk + j + e;
        if (sc > bv || (sc == bv && idx < bi)) { bv = sc; bi = idx; }
      }
    }
  }
  best = min(bi, 127);  // a row of NaNs has no maximum: stay inside the chunk
  best_v = bi == 0x7fffffff ? 0.f : bv;
}

// bf16 bit pattern of one exact 8-bit piece of a degree (piece 0: bits 0-7, 1: bits 8-15, 2: bits 16-23)
__device__ __forceinline__ uint32_t deg_piece(int deg, int piece) {
  return __float_as_uint((float)(deg & (0xff << (8 * piece)))) >> 16;
}

// Eq. 5 for the 32 B tokens b0 .. b0 + 31 of the chunk, one tensor, in place: the centroids replace the B rows.
// tgt[i] = B index A token i merges into (255: it does not); deg = degrees [A tokens | B tokens] or null (all one);
// dsum = summed degree of every B token's cluster; n_pieces = 8-bit pieces the degrees of the chunk need.
template <int C>
__device__ __forceinline__ void merge_rows(uint32_t tile, int b0, const unsigned char* tgt, const int* deg, const int* dsum,
                                           int n_pieces, int lane) {
  constexpr int NA = GroupCfg<C>::kNA;
  constexpr int KS = NA / 16;  // k steps of the A part
  const int g = lane >> 2, t = lane & 3;
  // which 16 x 16 blocks (m tile, k step) of the A part of W hold an entry
  unsigned need = 0;
#pragma unroll
  for (int m = 0; m < NA / 32; ++m) {
    const int i = lane + 32 * m, d = (int)tgt[i] - b0;
    if (d >= 0 && d < 32) need |= 1u << ((d >> 4) * KS + (i >> 4));
  }
  need = __reduce_or_sync(0xffffffffu, need);
  float inv[2][2];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) inv[mt][hi] = 1.0f / (float)dsum[b0 + 16 * mt + 8 * hi + g];
  const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8, k_c = lane >> 4;

#pragma unroll 1
  for (int h = 0; h < 2; ++h) {  // columns 64 h .. + 63: n tile j = columns 8 j .. + 7 of the half
    float acc[2][8][4];
    // the B tokens' own terms first: block (m tile mt, B tokens b0 + 16 mt ...) is a diagonal and starts the sums
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      uint32_t fb[4][4];
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) ldsm_x4_trans(g_addr<C>(tile, NA + b0 + 16 * mt + k_row, 8 * h + 2 * jp + k_c), fb[jp]);
      for (int piece = 0; piece < n_pieces; ++piece) {
        uint32_t w0 = kOneBits, w1 = kOneBits;
        if (deg) {
          w0 = deg_piece(deg[NA + b0 + 16 * mt + g], piece);
          w1 = deg_piece(deg[NA + b0 + 16 * mt + 8 + g], piece);
        }
        // row g of the diagonal block has its entry in column g: low half of the lane with 2t == g, high half of 2t + 1 == g
        const uint32_t d0 = (g == 2 * t) ? w0 : ((g == 2 * t + 1) ? (w0 << 16) : 0u);
        const uint32_t d1 = (g == 2 * t) ? w1 : ((g == 2 * t + 1) ? (w1 << 16) : 0u);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (piece == 0)
            mma_bf16_first(acc[mt][j], d0, 0u, 0u, d1, fb[j >> 1][2 * (j & 1)], fb[j >> 1][2 * (j & 1) + 1]);
          else
            mma_bf16(acc[mt][j], d0, 0u, 0u, d1, fb[j >> 1][2 * (j & 1)], fb[j >> 1][2 * (j & 1) + 1]);
        }
      }
    }
    // the A tokens that merge into these rows
#pragma unroll 1
    for (int ks = 0; ks < KS; ++ks) {
      if (!((need >> ks) & (1u | (1u << KS)))) continue;
      uint32_t fb[4][4];
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) ldsm_x4_trans(g_addr<C>(tile, 16 * ks + k_row, 8 * h + 2 * jp + k_c), fb[jp]);
      const int i0 = 16 * ks + 2 * t;  // A tokens i0, i0 + 1 (columns 2t, 2t + 1) and i0 + 8, i0 + 9
      const int tg0 = (int)tgt[i0] - b0, tg1 = (int)tgt[i0 + 1] - b0, tg2 = (int)tgt[i0 + 8] - b0, tg3 = (int)tgt[i0 + 9] - b0;
      for (int piece = 0; piece < n_pieces; ++piece) {
        uint32_t w0 = kOneBits, w1 = kOneBits << 16, w2 = kOneBits, w3 = kOneBits << 16;
        if (deg) {
          w0 = deg_piece(deg[i0], piece);
          w1 = deg_piece(deg[i0 + 1], piece) << 16;
          w2 = deg_piece(deg[i0 + 8], piece);
          w3 = deg_piece(deg[i0 + 9], piece) << 16;
        }
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
          if ((need >> (mt * KS + ks)) & 1u) {
            const int r = 16 * mt + g;
            const uint32_t a0 = (tg0 == r ? w0 : 0u) | (tg1 == r ? w1 : 0u), a1 = (tg0 == r + 8 ? w0 : 0u) | (tg1 == r + 8 ? w1 : 0u);
            const uint32_t a2 = (tg2 == r ? w2 : 0u) | (tg3 == r ? w3 : 0u), a3 = (tg2 == r + 8 ? w2 : 0u) | (tg3 == r + 8 ? w3 : 0u);
#pragma unroll
            for (int j = 0; j < 8; ++j) mma_bf16(acc[mt][j], a0, a1, a2, a3, fb[j >> 1][2 * (j & 1)], fb[j >> 1][2 * (j & 1) + 1]);
          }
      }
    }
    __syncwarp();  // every lane has read this warp's B rows of this half: they may be overwritten
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const float s = inv[mt][hi];
        uint32_t o[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          float x, y;
          mul_f32x2(x, y, acc[mt][j][2 * hi], acc[mt][j][2 * hi + 1], s);
          o[j] = pack_bf16x2(x, y);
        }
        const int row = NA + b0 + 16 * mt + 8 * hi + (lane & 7);
        stsm_x4(g_addr<C>(tile, row, 8 * h + (lane >> 3)), o[0], o[1], o[2], o[3]);
        stsm_x4(g_addr<C>(tile, row, 8 * h + 4 + (lane >> 3)), o[4], o[5], o[6], o[7]);
      }
  }
  __syncwarp();
}

// barrier among the warps of one group that also ORs a predicate over them
__device__ __forceinline__ bool group_or(int id, int threads, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %3, 0;\n\t"
      "bar.red.or.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(id), "r"(threads), "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}

template <int C, bool HAS_DEG>
__global__ void __launch_bounds__(GroupCfg<C>::kThreads, 1)
round_group_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ CUtensorMap tm_ko, const __grid_constant__ CUtensorMap tm_vo, const RoundArgs a,
                   const int n_full) {
  using Cfg = GroupCfg<C>;
  constexpr int NA = Cfg::kNA, GW = Cfg::kGW, GT = GW * 32;
  extern __shared__ __align__(1024) unsigned char smem[];
  griddep_wait();    // ordered launch: everything ahead in the stream has completed
  griddep_launch();  // the next launch may become resident as this grid's CTAs leave
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = warp / GW, w = warp % GW, gtid = w * 32 + lane, bar_id = 1 + grp;
  if ((smem_u32(smem) & 1023u) != 0u) {  // the swizzle pattern needs 1024-byte aligned tiles
    if (threadIdx.x == 0) atomicExch(a.status, 2);
    return;
  }
  const uint32_t tile = smem_u32(smem) + (uint32_t)grp * Cfg::kStage;
  unsigned char* extra = smem + (size_t)Cfg::kGroups * Cfg::kStage + (size_t)grp * Cfg::kExtra;
  int* deg = reinterpret_cast<int*>(extra + Cfg::oDeg);
  int* dsum = reinterpret_cast<int*>(extra + Cfg::oDsum);
  float* inv_b = reinterpret_cast<float*>(extra + Cfg::oInvB);
  float* simv = reinterpret_cast<float*>(extra + Cfg::oSim);
  int* newdeg = reinterpret_cast<int*>(extra + Cfg::oNewDeg);
  unsigned short* row_of = reinterpret_cast<unsigned short*>(extra + Cfg::oRowOf);
  unsigned char* tgt = extra + Cfg::oTgt;
  uint32_t* selmask = reinterpret_cast<uint32_t*>(extra + Cfg::oMask);
  const uint32_t bar = smem_u32(extra + Cfg::oBar), bar2 = smem_u32(extra + Cfg::oBar2);
  float* blk_inv = reinterpret_cast<float*>(extra + Cfg::oBlkInv);
  const int mode = a.mode;
  const bool every = mode == kModeAll, external = mode == kModeExternal;
  const bool umma = Cfg::kUmma && !external;  // (a pass that only merges computes no similarities)

  if (gtid == 0) {
    mbar_init(bar, 1);
    mbar_init(bar2, 1);
    mbar_init_fence();
  }
  if (umma && warp == 0) tmem_alloc(smem_u32(smem + Cfg::oTmem), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = umma ? *reinterpret_cast<volatile uint32_t*>(smem + Cfg::oTmem) : 0u;
  bool failed = false;

  const int64_t n_items = (int64_t)n_full * a.LH, stride = (int64_t)gridDim.x * Cfg::kGroups;
  int64_t item = (int64_t)blockIdx.x * Cfg::kGroups + grp;
  auto fetch = [&](const CUtensorMap* tm, int64_t it) {
    const int lh = (int)(it / n_full), ch = (int)(it - (int64_t)lh * n_full);
    mbar_arrive_expect_tx(bar, Cfg::kStage);
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int par = 0; par < 2; ++par) tma_load_4d(tile + h * Cfg::kHalf + par * (Cfg::kHalf / 2), tm, 64 * h, par, ch * NA, lh, bar);
  };
  auto sel_below = [&](int x) {  // selected A tokens with an index below x
    int cnt = 0;
#pragma unroll
    for (int m = 0; m < GW; ++m) {
      const int lim = x - 32 * m;
      const uint32_t bits = selmask[m];
      cnt += lim >= 32 ? __popc(bits) : (lim > 0 ? __popc(bits & ((1u << lim) - 1u)) : 0);
    }
    return cnt;
  };
  if (item < n_items && gtid == 0) fetch(&tm_k, item);

  uint32_t parity = 0;
  int n_done = 0;  // chunks this group has matched (the phase of bar2)
  for (; item < n_items; item += stride, ++n_done) {
    const int lh = (int)(item / n_full), ch = (int)(item - (int64_t)lh * n_full);
    const int64_t beg = a.lo + (int64_t)ch * C;
    const int64_t eslot = (int64_t)lh * a.edge_stride + (int64_t)ch * NA;
    const int64_t out_base = external ? (int64_t)a.chunk_out_off[(int64_t)lh * a.n_chunks + ch] : a.out_lo + (int64_t)ch * a.out_stride;
    int d_a = 1, d_b = 1, ext_b = -1, ext_sel = 0;
    if (HAS_DEG) {
      d_a = a.deg_src[(int64_t)lh * a.src_cap + beg + 2 * gtid];
      d_b = a.deg_src[(int64_t)lh * a.src_cap + beg + 2 * gtid + 1];
    }
    if (external) {
      ext_b = a.edge_b[eslot + gtid];
      ext_sel = a.sel[eslot + gtid];
    }
    // (the previous chunk's tables are free: its last reads lie before a group barrier or before this group's own waits)
    deg[gtid] = d_a;
    deg[NA + gtid] = d_b;
    dsum[gtid] = d_b;  // a cluster starts with its B token's own degree
    {
      const bool ok = mbar_wait(bar, parity);
      if (group_or(bar_id, GT, !ok)) {
        if (gtid == 0) atomicExch(a.status, 1);
        mbar_wait(bar, parity);  // the copies may still land: one more bounded wait before leaving
        failed = true;
        break;
      }
      parity ^= 1;
    }
    if (umma && gtid == 0) {
      // S = A B^T for the whole chunk: eight k steps of 16 columns (four per 64-column half of the tile)
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint32_t off = (uint32_t)(ks >> 2) * Cfg::kHalf + (uint32_t)(ks & 3) * 32u;
        umma_bf16(tmem + (uint32_t)grp * 128u, umma_desc_sw128(tile + off, 16, 1024),
                  umma_desc_sw128(tile + (uint32_t)NA * 128u + off, 16, 1024), group_idesc(), ks ? 1u : 0u);
      }
      umma_commit(bar2);
    }
    int n_pieces = 1;
    if (HAS_DEG) {
      const int dm = max(d_a, d_b);
      if (group_or(bar_id, GT, dm > 255)) n_pieces = group_or(bar_id, GT, dm > 65535) ? 3 : 2;
    }

    // ---- Sec. 5.2: one edge per A token
    int best = -1;
    float sim = 0.f;
    if (!external) {
      const float my_inv = inv_norms32<C>(tile, NA + 32 * w, lane);
      inv_b[gtid] = my_inv;
      if (Cfg::kUmma) {
        float m = my_inv;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) blk_inv[w] = m;
      }
      group_sync(bar_id, GT);
      if (Cfg::kUmma) {
        const bool ok = mbar_wait(bar2, (uint32_t)(n_done & 1));
        if (group_or(bar_id, GT, !ok)) {
          if (gtid == 0) atomicExch(a.status, 1);
          failed = true;
          break;
        }
        tc_fence_after();
        match_rows_tmem(tmem + ((uint32_t)(32 * w) << 16) + (uint32_t)grp * 128u, w, inv_b, blk_inv, best, sim);
        tc_fence_before();  // ordered before the group barriers below, behind which the next chunk's MMAs are issued
      } else {
        match_rows<C>(tile, 32 * w, inv_b, lane, best, sim);
      }
      if (mode == kModeChunkTopM) {
        sim *= inv_norms32<C>(tile, 32 * w, lane);  // Eq. 2: the ranking compares cosines
        simv[gtid] = sim;
        group_sync(bar_id, GT);
      }
    } else {
      best = ext_b >= 0 ? (ext_b >> 1) : -1;  // stored as the B token's local offset 2 b + 1
    }
    // ---- Sec. 5.3: which edges merge
    {
      bool s = best >= 0;
      if (mode == kModeChunkTopM) {
        int rank = 0;  // edges of this chunk ranked before mine: higher similarity, or equal and earlier
#pragma unroll 4
        for (int o = 0; o < NA; ++o) {
          const float other = simv[o];
          rank += (other > sim || (other == sim && o < gtid)) ? 1 : 0;
        }
        s = rank < a.m_full;
      } else if (external) {
        s = s && ext_sel != 0;
      }
      tgt[gtid] = s ? (unsigned char)best : (unsigned char)255;
      if (s) atomicAdd(&dsum[best], d_a);
      const uint32_t bits = __ballot_sync(0xffffffffu, s);
      if (lane == 0) selmask[w] = bits;
    }
    group_sync(bar_id, GT);

    // ---- output order: survivors keep their order, a merged A token shares its B token's slot
    int n_out = NA;
    if (every) {
      const int64_t di = (int64_t)lh * a.dst_cap + out_base + gtid;
      const int dg = dsum[gtid];
      a.deg_dst[di] = dg;
      if (a.logdeg_dst) a.logdeg_dst[di] = logf((float)dg);
      if (a.assign) {
        int32_t* as = a.assign + (int64_t)lh * a.assign_stride + beg;
        as[2 * gtid] = (int32_t)(out_base + tgt[gtid]);
        as[2 * gtid + 1] = (int32_t)(out_base + gtid);
      }
    } else {
      n_out = C - sel_below(NA);
      const int t_a = tgt[gtid];
      const int op_b = 2 * gtid + 1 - sel_below(gtid + 1);
      row_of[op_b] = (unsigned short)(NA + gtid);
      newdeg[op_b] = dsum[gtid];
      int op_a;
      if (t_a == 255) {
        op_a = 2 * gtid - sel_below(gtid);
        row_of[op_a] = (unsigned short)gtid;
        newdeg[op_a] = d_a;
      } else {
        op_a = 2 * t_a + 1 - sel_below(t_a + 1);
      }
      if (a.assign) {
        int32_t* as = a.assign + (int64_t)lh * a.assign_stride + beg;
        as[2 * gtid] = (int32_t)(out_base + op_a);
        as[2 * gtid + 1] = (int32_t)(out_base + op_b);
      }
    }

#pragma unroll 1
    for (int ph = 0; ph < 2; ++ph) {  // 0: keys (the tile that was matched), 1: values
      if (ph == 1) {
        const bool ok = mbar_wait(bar, parity);
        if (group_or(bar_id, GT, !ok)) {
          if (gtid == 0) atomicExch(a.status, 1);
          mbar_wait(bar, parity);
          failed = true;
          break;
        }
        parity ^= 1;
      }
      // ---- Eq. 5 for this warp's 32 B rows
      merge_rows<C>(tile, 32 * w, tgt, HAS_DEG ? deg : nullptr, dsum, n_pieces, lane);
      fence_async_smem();  // the TMA store reads the rows through the asynchronous proxy
      group_sync(bar_id, GT);
      if (every) {
        if (gtid == 0) {  // every A token merged: the B rows are the output, contiguous per half
          const CUtensorMap* tmo = ph == 0 ? &tm_ko : &tm_vo;
          tma_store_3d(tmo, 0, (int)out_base, lh, tile + NA * 128);
          tma_store_3d(tmo, 64, (int)out_base, lh, tile + Cfg::kHalf + NA * 128);
          bulk_commit();
          bulk_wait_read();  // the store has read the stage: the next tile may land in it
        }
      } else {
        unsigned char* dst = reinterpret_cast<unsigned char*>(ph == 0 ? a.k_dst : a.v_dst) + ((int64_t)lh * a.dst_cap + out_base) * 256;
        const int c16 = gtid & 15;
#pragma unroll 2
        for (int op = gtid >> 4; op < n_out; op += GT / 16) {
          uint4 x;
          ld_shared_v4(g_addr<C>(tile, row_of[op], c16), x);
          *reinterpret_cast<uint4*>(dst + (size_t)op * 256 + c16 * 16) = x;
        }
        if (ph == 0) {
          for (int op = gtid; op < n_out; op += GT) {
            const int64_t di = (int64_t)lh * a.dst_cap + out_base + op;
            const int dg = newdeg[op];
            a.deg_dst[di] = dg;
            if (a.logdeg_dst) a.logdeg_dst[di] = logf((float)dg);
          }
        }
        group_sync(bar_id, GT);  // every warp has copied its rows out of the stage
      }
      if (gtid == 0) {
        fence_async_smem();
        if (ph == 0)
          fetch(&tm_v, item);
        else if (item + stride < n_items)
          fetch(&tm_k, item + stride);
      }
    }
    if (failed) break;
  }
  if (umma) {  // every group is done with tensor memory
    tc_fence_before();
    if (__syncthreads_or(failed)) {
      // MMAs issued before the wait that gave up may still be running: they end on their own
      for (int i = 0; i < 1000; ++i) __nanosleep(1000);
      __syncthreads();
    }
    if (warp == 0) tmem_dealloc(tmem, 512);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn group_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// source view: (column 128, parity 2, token pair, slab) from token `lo` on; box = 64 columns of one parity for half a
// chunk's pairs, 128-byte swizzle
bool group_src_map(CUtensorMap* tm, const void* base, int64_t lo, int64_t pairs, int64_t cap, int LH, int box_pairs) {
  EncodeTiledFn fn = group_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {128, 2, (cuuint64_t)pairs, (cuuint64_t)LH};
  const cuuint64_t strides[3] = {256, 512, (cuuint64_t)cap * 256};
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)box_pairs, 1}, es[4] = {1, 1, 1, 1};
  void* addr = const_cast<unsigned char*>(static_cast<const unsigned char*>(base) + lo * 256);
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, addr, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// destination view: (column 128, row, slab); box = 64 columns x `rows` rows
bool group_dst_map(CUtensorMap* tm, void* base, int64_t cap, int LH, int rows) {
  EncodeTiledFn fn = group_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {128, (cuuint64_t)cap, (cuuint64_t)LH};
  const cuuint64_t strides[2] = {256, (cuuint64_t)cap * 256};
  const cuuint32_t box[3] = {64, (cuuint32_t)rows, 1}, es[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int C>
cudaError_t launch_group_c(const RoundArgs& a, int64_t n_full, cudaStream_t st) {
  using Cfg = GroupCfg<C>;
  CUtensorMap tm_k, tm_v, tm_ko, tm_vo;
  if (!group_src_map(&tm_k, a.k_src, a.lo, n_full * Cfg::kNA, a.src_cap, a.LH, Cfg::kNA) ||
      !group_src_map(&tm_v, a.v_src, a.lo, n_full * Cfg::kNA, a.src_cap, a.LH, Cfg::kNA) ||
      !group_dst_map(&tm_ko, a.k_dst, a.dst_cap, a.LH, Cfg::kNA) || !group_dst_map(&tm_vo, a.v_dst, a.dst_cap, a.LH, Cfg::kNA))
    return cudaErrorInvalidValue;
  const int64_t items = n_full * a.LH;
  const int64_t ctas = std::min<int64_t>(sm_count(), (items + Cfg::kGroups - 1) / Cfg::kGroups);
  auto kern = a.deg_src ? round_group_kernel<C, true> : round_group_kernel<C, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::kSmem);
  if (e != cudaSuccess) return e;
  return launch_dependent(kern, dim3((unsigned)ctas), dim3(Cfg::kThreads), Cfg::kSmem, st, tm_k, tm_v, tm_ko, tm_vo, a, (int)n_full);
}

}  // namespace

bool round_group_supported(const RoundArgs& a, int dtype, int D) {
  const bool merges = a.mode == kModeAll || a.mode == kModeChunkTopM || a.mode == kModeExternal;
  return dtype == 1 && D == 128 && (a.chunk == 128 || a.chunk == 256) && merges && a.status != nullptr && group_encode_fn() != nullptr &&
         (int64_t)a.LH * a.n_chunks < (1ll << 31);
}

// The full chunks of a round at chunk 128 / 256 in a mode that merges.  A shorter last chunk is left to the tile kernel.
cudaError_t launch_round_group(const RoundArgs& a, int64_t n_full, cudaStream_t st) {
  if (n_full <= 0) return cudaSuccess;
  return a.chunk == 256 ? launch_group_c<256>(a, n_full, st) : launch_group_c<128>(a, n_full, st);
}

}  // namespace ckv
