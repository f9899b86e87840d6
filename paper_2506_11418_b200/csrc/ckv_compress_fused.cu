// Two consecutive rounds of Chunked Soft Matching in one pass over the cache: bf16, chunk 64, head_dim 128, every
// edge merged in both rounds, source degrees all one (Algorithm 1's `while s > B` loop, first two iterations).
//
// Two neighbouring chunks of round 1 (128 tokens) leave 64 centroids, which are exactly one chunk of round 2 and
// leave 32 rows.  The intermediate cache of 64 rows per unit never goes to global memory: 512 bytes are read and
// 128 written per source token-vector instead of 768 + 384 for two separate passes.
//
// Persistent kernel, one CTA per SM, six groups of two warps, each group with one 32 KiB stage and its own mbarrier;
// the groups work on different units in different phases, the only barriers are named barriers inside a group.  A unit
// goes through its group's stage twice: first the K tile (matching of both rounds and the merged keys), then the V tile
// (the same clusters applied to the values).  Round 1 needs no exchange: warp w takes the unit's chunk w on its own and
// leaves its centroids over its own rows; round 2 is split by rows (16 A tokens and 16 output rows per warp) and
// exchanges targets and summed degrees through shared memory.
//   fetch     TMA tensor copies with 128-byte swizzle: a tile is two halves of 128 rows x 64 columns, so that both
//             row-wise (matching) and column-wise (merge) fragment loads are free of bank conflicts
//   Sec. 5.2  32 x 32 A x B dot products of a chunk on tensor cores (mma.sync m16n8k16, fp32 accumulate), squared
//             norms of the B keys from the diagonal of B B^T, row argmax of dot / |b| with the lowest index on ties
//   Eq. 5     the merge as a contraction C = W X: W [32 B tokens x 64 tokens] holds the degree of token k in row b
//             if k is b itself or an A token matched to b (degrees <= 33 here: exact in bf16), X is the staged tile
//             read column-wise; fp32 accumulate, times 1 / n', rounded to bf16 and written over the first rows of
//             the tile (16 x 16 blocks of W without an entry are skipped).  Rounding to bf16 between the rounds is
//             what a cache stored in bf16 between two separate rounds goes through
//   store     each warp sends the 16 final rows it produced: two TMA tensor stores per tensor
// Waits on the mbarrier are bounded: a warp that gives up records it in the status word and leaves.
#include <cuda.h>

#include <algorithm>
#include <cstdint>

#include "ckv_common.cuh"
#include "ckv_internal.h"
#include "ckv_ptx.cuh"

namespace ckv {

namespace {

using namespace ptx;

constexpr int kFGroups = 6;              // groups of two warps per CTA, each with its own stage
constexpr int kFThreads = kFGroups * 64;
constexpr int kFUnit = 128;              // source tokens per unit: two chunks of round 1
constexpr int kFHalf = kFUnit * 128;     // 128 rows x 64 columns (128 bytes each), swizzled
constexpr int kFStage = 2 * kFHalf;      // one tensor's tile of a unit: 32 KiB
constexpr int kFExtra = 512;             // per group: degrees after round 1 [64], after round 2 [32], round-2 targets [32], mbarrier
constexpr uint32_t kOneBf16 = 0x3f80u;   // 1.0
// Round 1 leaves the centroids where round 2 wants them: even positions (its A tokens) from row 0, odd positions (its B
// tokens) from row kFOdd.  (Row 68 instead of 64 would spread consecutive centroids over different banks for the
// matrix stores, but a base that is not a multiple of 8 costs more address arithmetic in every fragment load than the
// two-way conflicts of those few stores: measured 4.11 against 4.05 ms on the 131072-token workload.)
constexpr int kFOdd = 64;

struct FusedArgs {
  int32_t* deg_dst;
  float* logdeg_dst;     // may be null
  int32_t* assign1;      // may be null: [LH, stride1] slot of each source token after round 1
  int32_t* assign2;      // with assign1: [LH, stride2] slot of each round-1 slot after round 2
  int64_t stride1, stride2;
  int64_t dst_cap;
  int64_t lo;            // first token of the middle region (source, intermediate and final positions alike)
  uint32_t units;        // units per (layer, head)
  int64_t n_items;       // units * LH
  int32_t* status;
};

// byte address of 16-byte piece c16 (0..15) of row `row` of a swizzled tile
__device__ __forceinline__ uint32_t f_addr(uint32_t tile, int row, int c16) {
  return tile + (uint32_t)(c16 >> 3) * kFHalf + (uint32_t)row * 128u + (uint32_t)(((c16 & 7) ^ (row & 7)) << 4);
}

// Sec. 5.2 on one chunk: A tokens in rows row_a .. + 31 of the tile, B tokens in rows row_b .. + 31.  Returns, in lane
// i, the B index (0..31) that A token i is matched to.
__device__ __forceinline__ int match64(uint32_t tile, int row_a, int row_b, int lane) {
  const int g = lane >> 2, t = lane & 3;
  float acc[2][4][4];   // [m tile][n tile][c]: A token 16 mt + g (+8), B index 8 nt + 2t (+1)
  float nacc[2][2][4];  // B B^T diagonals
  // lane l supplies the address of row l % 8 of matrix l / 8.  A operand (16 tokens x 16 columns): matrices = (tokens
  // 0-7, 8-15) x (columns 0-7, 8-15) in the order a0 a1 a2 a3.  B operand of two n tiles: (tokens 0-7 | columns 0-7,
  // 8-15), then the next eight tokens: b0, b1 of n tile 2p, then of 2p + 1.
  const int a_row = row_a + (lane & 7) + ((lane >> 3) & 1) * 8, a_c = lane >> 4;
  const int b_row = row_b + (lane & 7) + (lane >> 4) * 8, b_c = (lane >> 3) & 1;
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {  // 16 columns per step
    uint32_t fa[2][4], fb[2][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) ldsm_x4(f_addr(tile, a_row + 16 * mt, 2 * kk + a_c), fa[mt]);
#pragma unroll
    for (int p = 0; p < 2; ++p) ldsm_x4(f_addr(tile, b_row + 16 * p, 2 * kk + b_c), fb[p]);
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const uint32_t b0 = fb[nt >> 1][2 * (nt & 1)], b1 = fb[nt >> 1][2 * (nt & 1) + 1];
        if (kk == 0)
          mma_bf16_first(acc[mt][nt], fa[mt][0], fa[mt][1], fa[mt][2], fa[mt][3], b0, b1);
        else
          mma_bf16(acc[mt][nt], fa[mt][0], fa[mt][1], fa[mt][2], fa[mt][3], b0, b1);
      }
    // B B^T on pairs of n tiles: rows = B indices 16 p + g (+8); the diagonal holds the squared norms
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      if (kk == 0) {
        mma_bf16_first(nacc[p][0], fb[p][0], fb[p][2], fb[p][1], fb[p][3], fb[p][0], fb[p][1]);
        mma_bf16_first(nacc[p][1], fb[p][0], fb[p][2], fb[p][1], fb[p][3], fb[p][2], fb[p][3]);
      } else {
        mma_bf16(nacc[p][0], fb[p][0], fb[p][2], fb[p][1], fb[p][3], fb[p][0], fb[p][1]);
        mma_bf16(nacc[p][1], fb[p][0], fb[p][2], fb[p][1], fb[p][3], fb[p][2], fb[p][3]);
      }
    }
  }
  // the squared norm of B index 8 nt + g sits on a diagonal: lane (g, t = g / 2), register g & 1 (+2 for odd nt)
  float inv0[4], inv1[4];
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) {
    const int p = nt >> 1, h = nt & 1;
    const float ss = (g & 1) ? nacc[p][h][2 * h + 1] : nacc[p][h][2 * h];
    const float inv = ss > 0.f ? rsqrtf(ss) : 0.f;          // a zero key has similarity 0 with everything
    inv0[nt] = __shfl_sync(0xffffffffu, inv, 9 * t);        // B index 8 nt + 2t     lives in lane 4 (2t) + t
    inv1[nt] = __shfl_sync(0xffffffffu, inv, 9 * t + 4);    // B index 8 nt + 2t + 1 lives in lane 4 (2t + 1) + t
  }
  // row argmax; dividing a row by |a| > 0 cannot change it
  int row_best[2][2];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      float bv = -INFINITY;
      int bi = 0x7fffffff;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const float s0 = acc[mt][nt][2 * hi] * inv0[nt] + 0.f, s1 = acc[mt][nt][2 * hi + 1] * inv1[nt] + 0.f;
        if (s0 > bv) { bv = s0; bi = 8 * nt + 2 * t; }
        if (s1 > bv) { bv = s1; bi = 8 * nt + 2 * t + 1; }
      }
#pragma unroll
      for (int o = 1; o <= 2; o <<= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      row_best[mt][hi] = bi;
    }
  // lane = A index i takes row i = 16 mt + 8 hi + g from the quad of g = i & 7
  int my_best = 0;
  const int src = 4 * (lane & 7), which = lane >> 3;
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      const int vb = __shfl_sync(0xffffffffu, row_best[mt][hi], src);
      if (which == 2 * mt + hi) my_best = vb;
    }
  return my_best & 31;  // a row of NaNs has no maximum: stay inside the chunk
}

// Eq. 5 on one chunk of one tensor, in place.  A tokens in rows row_a .. + 31, B tokens in rows row_b .. + 31; lane i
// holds the B index A token i merges into, lane j the summed degree n' of B token j's cluster.  deg_a / deg_b: degrees
// of the A and B tokens, element stride 2 (null: all one).  Centroid j goes to row dst0 + j (dst_split false) or, split
// by parity for the next round, to row dst0 + j / 2 (j even) / dst0 + kFOdd + j / 2 (j odd).
__device__ __forceinline__ void merge64(uint32_t tile, int row_a, int row_b, int dst0, bool dst_split, int my_best, int my_n,
                                        const int* deg_a, const int* deg_b, int lane) {
  const int g = lane >> 2, t = lane & 3;
  // W as the row-major A operand: rows = B index, columns = the chunk's tokens, A tokens first (k steps 0, 1), then B
  // tokens (k steps 2, 3).  The B tokens' own terms are the diagonal of blocks (m tile 0, step 2) and (1, 3); which
  // blocks of the A part hold an edge is found by a vote.
  const unsigned need = __reduce_or_sync(0xffffffffu, 1u << (((my_best >> 4) << 1) + (lane >> 4)));
  uint32_t wa[2][2][4];  // [m tile][k step][register]
#pragma unroll
  for (int ks = 0; ks < 2; ++ks) {
    const int i0 = 16 * ks + 2 * t;  // A tokens i0, i0 + 1 (columns 2t, 2t + 1) and i0 + 8, i0 + 9
    const int tg0 = __shfl_sync(0xffffffffu, my_best, i0), tg1 = __shfl_sync(0xffffffffu, my_best, i0 + 1);
    const int tg2 = __shfl_sync(0xffffffffu, my_best, i0 + 8), tg3 = __shfl_sync(0xffffffffu, my_best, i0 + 9);
    uint32_t w0 = kOneBf16, w1 = kOneBf16 << 16, w2 = kOneBf16, w3 = kOneBf16 << 16;
    if (deg_a) {  // degrees up to 256 are exact in bf16
      w0 = __float_as_uint((float)deg_a[2 * i0]) >> 16;
      w1 = __float_as_uint((float)deg_a[2 * i0 + 2]) & 0xffff0000u;
      w2 = __float_as_uint((float)deg_a[2 * i0 + 16]) >> 16;
      w3 = __float_as_uint((float)deg_a[2 * i0 + 18]) & 0xffff0000u;
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      const int r = 16 * mt + g;
      wa[mt][ks][0] = (tg0 == r ? w0 : 0u) | (tg1 == r ? w1 : 0u);
      wa[mt][ks][1] = (tg0 == r + 8 ? w0 : 0u) | (tg1 == r + 8 ? w1 : 0u);
      wa[mt][ks][2] = (tg2 == r ? w2 : 0u) | (tg3 == r ? w3 : 0u);
      wa[mt][ks][3] = (tg2 == r + 8 ? w2 : 0u) | (tg3 == r + 8 ? w3 : 0u);
    }
  }
  // own terms: row g of the diagonal block has its entry in column g: register 0 (rows 0-7) and 3 (rows 8-15) of the
  // lane with 2t == g (low half) or 2t + 1 == g (high half)
  uint32_t wd[2][2];  // [m tile][rows 0-7 / 8-15]
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      uint32_t w = kOneBf16;
      if (deg_b) w = __float_as_uint((float)deg_b[2 * (16 * mt + 8 * hi + g)]) >> 16;
      wd[mt][hi] = (g == 2 * t) ? w : ((g == 2 * t + 1) ? (w << 16) : 0u);
    }
  const float my_inv = 1.0f / (float)my_n;
  float inv[2][2];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) inv[mt][hi] = __shfl_sync(0xffffffffu, my_inv, 16 * mt + 8 * hi + g);

  // ldmatrix.trans: lane l supplies row l % 8 (+8 for odd l / 8) of the sixteen tokens of a k step, 16-byte piece
  // 2 jp + l / 16 -> b0, b1 of n tile 2 jp, then of 2 jp + 1.  stmatrix: row l % 8 of the eight output rows, piece l / 8.
  const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8, k_c = lane >> 4;
#pragma unroll 1
  for (int h = 0; h < 2; ++h) {  // columns 64 h .. + 63: n tile j = columns 8 j .. + 7 of the half
    float acc[2][8][4];
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      const int step = (ks + 2) & 3;  // the B tokens first (steps 2, 3): their blocks are always there and start the sums
      if (step < 2 && !((need >> step) & 5u)) continue;
      const int base = step < 2 ? row_a + 16 * step : row_b + 16 * (step - 2);
      uint32_t fb[4][4];
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) ldsm_x4_trans(f_addr(tile, base + k_row, 8 * h + 2 * jp + k_c), fb[jp]);
      if (step >= 2) {
        const int mt = step - 2;
#pragma unroll
        for (int j = 0; j < 8; ++j)
          mma_bf16_first(acc[mt][j], wd[mt][0], 0u, 0u, wd[mt][1], fb[j >> 1][2 * (j & 1)], fb[j >> 1][2 * (j & 1) + 1]);
      } else {
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
          if ((need >> (2 * mt + step)) & 1u) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              mma_bf16(acc[mt][j], wa[mt][step][0], wa[mt][step][1], wa[mt][step][2], wa[mt][step][3], fb[j >> 1][2 * (j & 1)],
                       fb[j >> 1][2 * (j & 1) + 1]);
          }
      }
    }
    __syncwarp();  // every lane has read this half's rows: they may be overwritten
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
        const int j_out = 16 * mt + 8 * hi + (lane & 7);
        const int row = dst_split ? dst0 + (j_out & 1) * kFOdd + (j_out >> 1) : dst0 + j_out;
        stsm_x4(f_addr(tile, row, 8 * h + (lane >> 3)), o[0], o[1], o[2], o[3]);
        stsm_x4(f_addr(tile, row, 8 * h + 4 + (lane >> 3)), o[4], o[5], o[6], o[7]);
      }
  }
  __syncwarp();
}

// ---- round 2, split between the two warps of a group.  Its chunk are the 64 centroids of round 1: A tokens (even
// positions) i = 0..31 in rows 32 (i / 16) + i % 16, B tokens in rows 64 + the same (each warp left its chunk's centroids
// over its own rows), degrees d1[2 i] and d1[2 i + 1].

__device__ __forceinline__ void group_sync2(int id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }

__device__ __forceinline__ bool group_or2(int id, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %2, 0;\n\t"
      "bar.red.or.pred p, %1, 64, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(id), "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}

// Sec. 5.2 for the 16 A tokens 16 w .. 16 w + 15 of the round-2 chunk against its 32 B tokens: writes each one's target
// to tgt2 and adds its degree to the target's summed degree.
__device__ __forceinline__ void match2(uint32_t tile, int w, unsigned char* tgt2, int* dsum2, const int* d1, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const int a_row = 32 * w + (lane & 7) + ((lane >> 3) & 1) * 8, a_c = lane >> 4;
  const int b_row = 64 + (lane & 7) + (lane >> 4) * 8, b_c = (lane >> 3) & 1;  // + 32 p: B tokens 16 p .. 16 p + 15
  float acc[4][4];      // [n tile][c]: A token 16 w + g (+8), B index 8 nt + 2t (+1)
  float nacc[2][2][4];  // B B^T diagonals
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    uint32_t fa[4], fb[2][4];
    ldsm_x4(f_addr(tile, a_row, 2 * kk + a_c), fa);
#pragma unroll
    for (int p = 0; p < 2; ++p) ldsm_x4(f_addr(tile, b_row + 32 * p, 2 * kk + b_c), fb[p]);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const uint32_t b0 = fb[nt >> 1][2 * (nt & 1)], b1 = fb[nt >> 1][2 * (nt & 1) + 1];
      if (kk == 0)
        mma_bf16_first(acc[nt], fa[0], fa[1], fa[2], fa[3], b0, b1);
      else
        mma_bf16(acc[nt], fa[0], fa[1], fa[2], fa[3], b0, b1);
    }
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      if (kk == 0) {
        mma_bf16_first(nacc[p][0], fb[p][0], fb[p][2], fb[p][1], fb[p][3], fb[p][0], fb[p][1]);
        mma_bf16_first(nacc[p][1], fb[p][0], fb[p][2], fb[p][1], fb[p][3], fb[p][2], fb[p][3]);
      } else {
        mma_bf16(nacc[p][0], fb[p][0], fb[p][2], fb[p][1], fb[p][3], fb[p][0], fb[p][1]);
        mma_bf16(nacc[p][1], fb[p][0], fb[p][2], fb[p][1], fb[p][3], fb[p][2], fb[p][3]);
      }
    }
  }
  float inv0[4], inv1[4];
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) {
    const int p = nt >> 1, h = nt & 1;
    const float ss = (g & 1) ? nacc[p][h][2 * h + 1] : nacc[p][h][2 * h];
    const float inv = ss > 0.f ? rsqrtf(ss) : 0.f;
    inv0[nt] = __shfl_sync(0xffffffffu, inv, 9 * t);
    inv1[nt] = __shfl_sync(0xffffffffu, inv, 9 * t + 4);
  }
#pragma unroll
  for (int hi = 0; hi < 2; ++hi) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const float s0 = acc[nt][2 * hi] * inv0[nt] + 0.f, s1 = acc[nt][2 * hi + 1] * inv1[nt] + 0.f;
      if (s0 > bv) { bv = s0; bi = 8 * nt + 2 * t; }
      if (s1 > bv) { bv = s1; bi = 8 * nt + 2 * t + 1; }
    }
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (t == 0) {
      const int i2 = 16 * w + 8 * hi + g;
      bi &= 31;  // a row of NaNs has no maximum: stay inside the chunk
      tgt2[i2] = (unsigned char)bi;
      atomicAdd(&dsum2[bi], d1[2 * i2]);
    }
  }
}

// Eq. 5 for the 16 B tokens 16 w .. 16 w + 15 of the round-2 chunk, one tensor: the final rows go to rows
// 16 + 32 w .. of the tile, which nobody reads any more.
__device__ __forceinline__ void merge2(uint32_t tile, int w, const unsigned char* tgt2, const int* d1, const int* dsum2, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const int dt = (int)tgt2[lane] - 16 * w;
  const unsigned need = __reduce_or_sync(0xffffffffu, (dt >= 0 && dt < 16) ? 1u << (lane >> 4) : 0u);  // k steps of the A part in use
  const uint32_t wd0 = __float_as_uint((float)d1[2 * (16 * w + g) + 1]) >> 16, wd1 = __float_as_uint((float)d1[2 * (16 * w + 8 + g) + 1]) >> 16;
  const uint32_t dg0 = (g == 2 * t) ? wd0 : ((g == 2 * t + 1) ? (wd0 << 16) : 0u);
  const uint32_t dg1 = (g == 2 * t) ? wd1 : ((g == 2 * t + 1) ? (wd1 << 16) : 0u);
  uint32_t wa[2][4];
#pragma unroll
  for (int ks = 0; ks < 2; ++ks) {
    const int i0 = 16 * ks + 2 * t;
    const int tg0 = (int)tgt2[i0] - 16 * w, tg1 = (int)tgt2[i0 + 1] - 16 * w, tg2 = (int)tgt2[i0 + 8] - 16 * w, tg3 = (int)tgt2[i0 + 9] - 16 * w;
    const uint32_t w0 = __float_as_uint((float)d1[2 * i0]) >> 16, w1 = __float_as_uint((float)d1[2 * i0 + 2]) & 0xffff0000u;
    const uint32_t w2 = __float_as_uint((float)d1[2 * i0 + 16]) >> 16, w3 = __float_as_uint((float)d1[2 * i0 + 18]) & 0xffff0000u;
    wa[ks][0] = (tg0 == g ? w0 : 0u) | (tg1 == g ? w1 : 0u);
    wa[ks][1] = (tg0 == g + 8 ? w0 : 0u) | (tg1 == g + 8 ? w1 : 0u);
    wa[ks][2] = (tg2 == g ? w2 : 0u) | (tg3 == g ? w3 : 0u);
    wa[ks][3] = (tg2 == g + 8 ? w2 : 0u) | (tg3 == g + 8 ? w3 : 0u);
  }
  const float inv0 = 1.0f / (float)dsum2[16 * w + g], inv1 = 1.0f / (float)dsum2[16 * w + 8 + g];
  const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8, k_c = lane >> 4;
#pragma unroll 1
  for (int h = 0; h < 2; ++h) {
    float acc[8][4];
    {
      uint32_t fb[4][4];  // the B tokens' own rows: the diagonal block starts the sums
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) ldsm_x4_trans(f_addr(tile, 64 + 32 * w + k_row, 8 * h + 2 * jp + k_c), fb[jp]);
#pragma unroll
      for (int j = 0; j < 8; ++j) mma_bf16_first(acc[j], dg0, 0u, 0u, dg1, fb[j >> 1][2 * (j & 1)], fb[j >> 1][2 * (j & 1) + 1]);
    }
#pragma unroll
    for (int ks = 0; ks < 2; ++ks)
      if ((need >> ks) & 1u) {
        uint32_t fb[4][4];
#pragma unroll
        for (int jp = 0; jp < 4; ++jp) ldsm_x4_trans(f_addr(tile, 32 * ks + k_row, 8 * h + 2 * jp + k_c), fb[jp]);
#pragma unroll
        for (int j = 0; j < 8; ++j) mma_bf16(acc[j], wa[ks][0], wa[ks][1], wa[ks][2], wa[ks][3], fb[j >> 1][2 * (j & 1)], fb[j >> 1][2 * (j & 1) + 1]);
      }
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      const float sc = hi ? inv1 : inv0;
      uint32_t o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float x, y;
        mul_f32x2(x, y, acc[j][2 * hi], acc[j][2 * hi + 1], sc);
        o[j] = pack_bf16x2(x, y);
      }
      const int row = 16 + 32 * w + 8 * hi + (lane & 7);
      stsm_x4(f_addr(tile, row, 8 * h + (lane >> 3)), o[0], o[1], o[2], o[3]);
      stsm_x4(f_addr(tile, row, 8 * h + 4 + (lane >> 3)), o[4], o[5], o[6], o[7]);
    }
  }
  __syncwarp();
}

__global__ void __launch_bounds__(kFThreads, 1)
round_fused2_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    const __grid_constant__ CUtensorMap tm_ko, const __grid_constant__ CUtensorMap tm_vo, const FusedArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  griddep_wait();    // ordered launch: everything ahead in the stream has completed
  griddep_launch();  // the next launch may become resident as this grid's CTAs leave
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = warp >> 1, w = warp & 1, gtid = 32 * w + lane, bar_id = 1 + grp;
  if ((smem_u32(smem) & 1023u) != 0u) {  // the swizzle pattern needs 1024-byte aligned tiles
    if (threadIdx.x == 0) atomicExch(a.status, 2);
    return;
  }
  const uint32_t tile = smem_u32(smem) + (uint32_t)grp * kFStage;
  unsigned char* extra = smem + (size_t)kFGroups * kFStage + (size_t)grp * kFExtra;
  int* d1 = reinterpret_cast<int*>(extra);          // [64] degrees after round 1, in the order of the round-2 chunk
  int* dsum2 = reinterpret_cast<int*>(extra + 256);  // [32] degrees after round 2
  unsigned char* tgt2 = extra + 384;                 // [32] round-2 targets
  const uint32_t bar = smem_u32(extra + 416);

  if (gtid == 0) {
    mbar_init(bar, 1);
    mbar_init_fence();
  }
  __syncthreads();

  const int64_t stride = (int64_t)gridDim.x * kFGroups;
  int64_t item = (int64_t)blockIdx.x * kFGroups + grp;
  // a tile: per half of the columns, the unit's 64 A tokens (1st, 3rd, ... token) in rows 0-63, its B tokens in 64-127
  auto fetch = [&](const CUtensorMap* tm, int64_t it) {
    const uint32_t lh = (uint32_t)it / a.units, u = (uint32_t)it - lh * a.units;
    const int pair = (int)(u * (kFUnit / 2));
    mbar_arrive_expect_tx(bar, kFStage);
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int par = 0; par < 2; ++par) tma_load_4d(tile + h * kFHalf + par * (kFHalf / 2), tm, 64 * h, par, pair, (int)lh, bar);
  };
  if (item < a.n_items && gtid == 0) fetch(&tm_k, item);

  uint32_t parity = 0;
  for (; item < a.n_items; item += stride) {
    const uint32_t lh = (uint32_t)item / a.units, u = (uint32_t)item - lh * a.units;
    const int out_row = (int)(a.lo + (int64_t)u * 32);
    int best1 = 0, n1 = 1;  // round 1, this warp's chunk: lane i = A token i's target, lane j = B token j's summed degree
#pragma unroll 1
    for (int ph = 0; ph < 2; ++ph) {  // 0: the K tile (matching and merged keys), 1: the V tile (the same clusters)
      const bool ok = mbar_wait(bar, parity);
      if (group_or2(bar_id, !ok)) {
        if (gtid == 0) atomicExch(a.status, 1);
        mbar_wait(bar, parity);  // the copies may still land: one more bounded wait before leaving
        return;
      }
      parity ^= 1;
      // ---- round 1: warp w on the unit's chunk w, on its own
      if (ph == 0) {
        best1 = match64(tile, 32 * w, 64 + 32 * w, lane);
        d1[32 * w + lane] = 1;
        __syncwarp();
        atomicAdd(&d1[32 * w + best1], 1);
        __syncwarp();
        n1 = d1[32 * w + lane];
      }
      // centroid j of chunk w lands where round 2 finds it: A tokens of round 2 over this chunk's A rows, B tokens over its B rows
      merge64(tile, 32 * w, 64 + 32 * w, 32 * w, true, best1, n1, nullptr, nullptr, lane);
      group_sync2(bar_id);  // both chunks' centroids and degrees are in place
      // ---- round 2 on the 64 centroids
      if (ph == 0) {
        if (gtid < 32) dsum2[gtid] = d1[2 * gtid + 1];  // a cluster starts with its B token's own degree
        group_sync2(bar_id);
        match2(tile, w, tgt2, dsum2, d1, lane);
        group_sync2(bar_id);  // targets and summed degrees of the whole chunk
        if (gtid < 32) {
          const int64_t di = (int64_t)lh * a.dst_cap + out_row + gtid;
          const int dg = dsum2[gtid];
          a.deg_dst[di] = dg;
          if (a.logdeg_dst) a.logdeg_dst[di] = logf((float)dg);
        }
        if (a.assign1) {
          // round 1: token -> intermediate slot; round 2: intermediate slot -> final slot (composed by the caller)
          const int s1 = (int)(a.lo + (int64_t)u * 64);
          int32_t* as1 = a.assign1 + (int64_t)lh * a.stride1 + a.lo + (int64_t)u * kFUnit + 64 * w;
          as1[2 * lane] = s1 + 32 * w + best1;
          as1[2 * lane + 1] = s1 + 32 * w + lane;
          if (w == 0) {
            int32_t* as2 = a.assign2 + (int64_t)lh * a.stride2 + s1;
            as2[2 * lane] = out_row + tgt2[lane];
            as2[2 * lane + 1] = out_row + lane;
          }
        }
      }
      merge2(tile, w, tgt2, d1, dsum2, lane);
      fence_async_smem();  // the TMA store reads the rows through the asynchronous proxy
      __syncwarp();
      if (lane == 0) {  // each warp stores the 16 final rows it produced
        const CUtensorMap* tmo = ph == 0 ? &tm_ko : &tm_vo;
        tma_store_3d(tmo, 0, out_row + 16 * w, (int)lh, tile + (16 + 32 * w) * 128);
        tma_store_3d(tmo, 64, out_row + 16 * w, (int)lh, tile + kFHalf + (16 + 32 * w) * 128);
        bulk_commit();
        bulk_wait_read();
      }
      group_sync2(bar_id);  // both stores have read the stage, nobody reads it any more: the next tile may land
      if (gtid == 0) {
        fence_async_smem();
        if (ph == 0)
          fetch(&tm_v, item);
        else if (item + stride < a.n_items)
          fetch(&tm_k, item + stride);
      }
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn fused_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// source view: (column 128, parity 2, token pair, slab) from token `lo` on; box = 64 columns of one parity for 64
// pairs, 128-byte swizzle: the A tokens and the B tokens of a unit land in separate runs of rows
bool make_src_map(CUtensorMap* tm, const void* base, int64_t lo, int64_t pairs, int64_t cap, int LH) {
  EncodeTiledFn fn = fused_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {128, 2, (cuuint64_t)pairs, (cuuint64_t)LH};
  const cuuint64_t strides[3] = {256, 512, (cuuint64_t)cap * 256};
  const cuuint32_t box[4] = {64, 1, kFUnit / 2, 1}, es[4] = {1, 1, 1, 1};
  void* addr = const_cast<unsigned char*>(static_cast<const unsigned char*>(base) + lo * 256);
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, addr, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// (column 128, token, slab) view of a cache; box = 64 columns x `rows` tokens, 128-byte swizzle
bool make_map(CUtensorMap* tm, const void* base, int64_t cap, int LH, int rows, bool load) {
  EncodeTiledFn fn = fused_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {128, (cuuint64_t)cap, (cuuint64_t)LH};
  const cuuint64_t strides[2] = {256, (cuuint64_t)cap * 256};
  const cuuint32_t box[3] = {64, (cuuint32_t)rows, 1}, es[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, load ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool round_fused2_supported(int dtype, int D, int chunk) {
  return dtype == 1 && D == 128 && chunk == 64 && fused_encode_fn() != nullptr;
}

// Rounds j and j + 1 of a schedule on the first 2 * units chunks of every slab: a.k_src / a.v_src (degrees all one)
// -> a.k_dst / a.v_dst, a.deg_dst, a.logdeg_dst.  assign1 / assign2: a.assign with a.assign_stride, and step2.
cudaError_t launch_round_fused2(const RoundArgs& r, int64_t units, int32_t* assign2, int64_t stride2, cudaStream_t st) {
  if (units <= 0) return cudaSuccess;
  CUtensorMap tm_k, tm_v, tm_ko, tm_vo;
  if (!make_src_map(&tm_k, r.k_src, r.lo, units * (kFUnit / 2), r.src_cap, r.LH) ||
      !make_src_map(&tm_v, r.v_src, r.lo, units * (kFUnit / 2), r.src_cap, r.LH) ||
      !make_map(&tm_ko, r.k_dst, r.dst_cap, r.LH, 16, false) || !make_map(&tm_vo, r.v_dst, r.dst_cap, r.LH, 16, false))
    return cudaErrorInvalidValue;
  FusedArgs a{};
  a.deg_dst = r.deg_dst;
  a.logdeg_dst = r.logdeg_dst;
  a.assign1 = r.assign;
  a.assign2 = r.assign ? assign2 : nullptr;
  a.stride1 = r.assign_stride;
  a.stride2 = stride2;
  a.dst_cap = r.dst_cap;
  a.lo = r.lo;
  a.units = (uint32_t)units;
  a.n_items = units * r.LH;
  a.status = r.status;
  const size_t smem = (size_t)kFGroups * (kFStage + kFExtra);
  cudaError_t e = cudaFuncSetAttribute(round_fused2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int64_t ctas = std::min<int64_t>(sm_count(), (a.n_items + kFGroups - 1) / kFGroups);
  return launch_dependent(round_fused2_kernel, dim3((unsigned)ctas), dim3(kFThreads), smem, st, tm_k, tm_v, tm_ko, tm_vo, a);
}

}  // namespace ckv
