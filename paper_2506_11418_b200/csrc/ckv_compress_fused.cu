// Two consecutive rounds of Chunked Soft Matching in one pass over the cache: bf16, chunk 64, head_dim 128, every
// edge merged in both rounds, source degrees all one (Algorithm 1's `while s > B` loop, first two iterations).
//
// Two neighbouring chunks of round 1 (128 tokens) leave 64 centroids, which are exactly one chunk of round 2 and
// leave 32 rows.  The intermediate cache of 64 rows per unit never goes to global memory: 512 bytes are read and
// 128 written per source token-vector instead of 768 + 384 for two separate passes.
//
// Persistent kernel, one CTA per SM, every warp an independent worker with one 32 KiB stage and its own mbarrier.
// A worker handles a unit in two phases through the same stage: first the K tile (matching of both rounds and the
// merged keys), then the V tile (the same clusters applied to the values).
//   fetch     TMA tensor copies with 128-byte swizzle: a tile is two halves of 128 rows x 64 columns, so that both
//             row-wise (matching) and column-wise (merge) fragment loads are free of bank conflicts
//   Sec. 5.2  32 x 32 A x B dot products of a chunk on tensor cores (mma.sync m16n8k16, fp32 accumulate), squared
//             norms of the B keys from the diagonal of B B^T, row argmax of dot / |b| with the lowest index on ties
//   Eq. 5     the merge as a contraction C = W X: W [32 B tokens x 64 tokens] holds the degree of token k in row b
//             if k is b itself or an A token matched to b (degrees <= 33 here: exact in bf16), X is the staged tile
//             read column-wise; fp32 accumulate, times 1 / n', rounded to bf16 and written over the first rows of
//             the tile (16 x 16 blocks of W without an entry are skipped).  Rounding to bf16 between the rounds is
//             what a cache stored in bf16 between two separate rounds goes through
//   store     the 32 final rows of a unit leave as two TMA tensor stores per tensor
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

constexpr int kFWarps = 7;
constexpr int kFUnit = 128;              // source tokens per unit: two chunks of round 1
constexpr int kFHalf = kFUnit * 128;     // 128 rows x 64 columns (128 bytes each), swizzled
constexpr int kFStage = 2 * kFHalf;      // one tensor's tile of a unit: 32 KiB
constexpr int kFExtra = 400;             // per warp: degrees after round 1 [64], after round 2 [32], mbarrier, pad
constexpr uint32_t kOneBf16 = 0x3f80u;   // 1.0

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

// Sec. 5.2 on one chunk (rows row0 .. row0 + 63 of the tile; A = even rows, B = odd rows): returns, in lane i, the
// B index (0..31) that A token i is matched to.
__device__ __forceinline__ int match64(uint32_t tile, int row0, int lane) {
  const int g = lane >> 2, t = lane & 3;
  float acc[2][4][4];   // [m tile][n tile][c]: A token 16 mt + g (+8), B index 8 nt + 2t (+1)
  float nacc[2][2][4];  // B B^T diagonals
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[i][j][c] = 0.f;
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int c = 0; c < 4; ++c) nacc[i][j][c] = 0.f;

#pragma unroll
  for (int kp = 0; kp < 4; ++kp) {
    // each lane reads 16 contiguous bytes of a row (elements 32 kp + 8 t .. + 7); the same permutation of the
    // contraction index on both operands leaves the dot products unchanged
    const int c16 = 4 * kp + t;
    uint4 ra[2][2], rb[4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) ld_shared_v4(f_addr(tile, row0 + 2 * (16 * mt + 8 * hi + g), c16), ra[mt][hi]);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) ld_shared_v4(f_addr(tile, row0 + 2 * (8 * nt + g) + 1, c16), rb[nt]);
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
      uint32_t b0[4], b1[4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        b0[nt] = ks ? rb[nt].z : rb[nt].x;
        b1[nt] = ks ? rb[nt].w : rb[nt].y;
      }
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const uint32_t a0 = ks ? ra[mt][0].z : ra[mt][0].x, a1 = ks ? ra[mt][1].z : ra[mt][1].x;
        const uint32_t a2 = ks ? ra[mt][0].w : ra[mt][0].y, a3 = ks ? ra[mt][1].w : ra[mt][1].y;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) mma_bf16(acc[mt][nt], a0, a1, a2, a3, b0[nt], b1[nt]);
      }
      // B B^T on pairs of n tiles: rows = B indices 16 p + g (+8); the diagonal holds the squared norms
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        mma_bf16(nacc[p][0], b0[2 * p], b0[2 * p + 1], b1[2 * p], b1[2 * p + 1], b0[2 * p], b1[2 * p]);
        mma_bf16(nacc[p][1], b0[2 * p], b0[2 * p + 1], b1[2 * p], b1[2 * p + 1], b0[2 * p + 1], b1[2 * p + 1]);
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
  int row_b[2][2];
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
      row_b[mt][hi] = bi;
    }
  // lane = A index i takes row i = 16 mt + 8 hi + g from the quad of g = i & 7
  int my_best = 0;
  const int src = 4 * (lane & 7), which = lane >> 3;
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      const int vb = __shfl_sync(0xffffffffu, row_b[mt][hi], src);
      if (which == 2 * mt + hi) my_best = vb;
    }
  return my_best & 31;  // a row of NaNs has no maximum: stay inside the chunk
}

// Eq. 5 on one chunk of one tensor, in place: tokens = rows src_row0 .. + 63 of the tile (A = even, B = odd), lane i
// holds the B index A token i merges into; the 32 centroids go to rows dst_row0 .. + 31.  deg_in: the 64 tokens'
// degrees (null: all one); deg_out: the 32 summed degrees.
__device__ __forceinline__ void merge64(uint32_t tile, int src_row0, int dst_row0, int my_best, const int* deg_in,
                                        const int* deg_out, int lane) {
  const int g = lane >> 2, t = lane & 3;
  // which 16 x 16 blocks (m tile, k step) of W hold an entry: the B tokens' own terms, and the edges
  const unsigned need = __reduce_or_sync(0xffffffffu, 1u << (((my_best >> 4) << 2) + (lane >> 3))) | 0xc3u;
  // W as the row-major A operand: rows = B index, columns = token of the chunk
  uint32_t wf[2][4][4];
#pragma unroll
  for (int ks = 0; ks < 4; ++ks) {
    const int i0 = 8 * ks + t, i1 = i0 + 4;  // A token i (token 2i) and B token i (token 2i + 1) share a register
    const int tg0 = __shfl_sync(0xffffffffu, my_best, i0), tg1 = __shfl_sync(0xffffffffu, my_best, i1);
    uint32_t wa0 = kOneBf16, wb0 = kOneBf16 << 16, wa1 = kOneBf16, wb1 = kOneBf16 << 16;
    if (deg_in) {
      wa0 = __float_as_uint((float)deg_in[2 * i0]) >> 16;
      wb0 = __float_as_uint((float)deg_in[2 * i0 + 1]) & 0xffff0000u;
      wa1 = __float_as_uint((float)deg_in[2 * i1]) >> 16;
      wb1 = __float_as_uint((float)deg_in[2 * i1 + 1]) & 0xffff0000u;
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      const int r = 16 * mt + g;
      wf[mt][ks][0] = (tg0 == r ? wa0 : 0u) | (i0 == r ? wb0 : 0u);
      wf[mt][ks][1] = (tg0 == r + 8 ? wa0 : 0u) | (i0 == r + 8 ? wb0 : 0u);
      wf[mt][ks][2] = (tg1 == r ? wa1 : 0u) | (i1 == r ? wb1 : 0u);
      wf[mt][ks][3] = (tg1 == r + 8 ? wa1 : 0u) | (i1 == r + 8 ? wb1 : 0u);
    }
  }
  float inv[2][2];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) inv[mt][hi] = 1.0f / (float)deg_out[16 * mt + 8 * hi + g];

#pragma unroll 1
  for (int h = 0; h < 2; ++h) {
    // columns 64 h .. + 63.  n tile j, column n = g  <->  tile column 64 h + 8 g + j: a lane's 16-byte piece feeds
    // eight n tiles, and an accumulator row ends up with 16 contiguous columns per lane
    float acc[2][8][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[mt][j][c] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      const int r0 = src_row0 + 16 * ks + 2 * t;
      uint4 x[4];
      ld_shared_v4(f_addr(tile, r0, 8 * h + g), x[0]);
      ld_shared_v4(f_addr(tile, r0 + 1, 8 * h + g), x[1]);
      ld_shared_v4(f_addr(tile, r0 + 8, 8 * h + g), x[2]);
      ld_shared_v4(f_addr(tile, r0 + 9, 8 * h + g), x[3]);
      const uint32_t x0[4] = {x[0].x, x[0].y, x[0].z, x[0].w}, x1[4] = {x[1].x, x[1].y, x[1].z, x[1].w};
      const uint32_t x2[4] = {x[2].x, x[2].y, x[2].z, x[2].w}, x3[4] = {x[3].x, x[3].y, x[3].z, x[3].w};
      uint32_t b0[8], b1[8];  // (token 2t, token 2t + 1) and (token 2t + 8, token 2t + 9) of column 8 g + j
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        b0[2 * w] = __byte_perm(x0[w], x1[w], 0x5410);
        b0[2 * w + 1] = __byte_perm(x0[w], x1[w], 0x7632);
        b1[2 * w] = __byte_perm(x2[w], x3[w], 0x5410);
        b1[2 * w + 1] = __byte_perm(x2[w], x3[w], 0x7632);
      }
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
        if ((need >> (4 * mt + ks)) & 1u) {
#pragma unroll
          for (int j = 0; j < 8; ++j) mma_bf16(acc[mt][j], wf[mt][ks][0], wf[mt][ks][1], wf[mt][ks][2], wf[mt][ks][3], b0[j], b1[j]);
        }
    }
    __syncwarp();  // every lane has read this half's rows: they may be overwritten
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const int row = dst_row0 + 16 * mt + 8 * hi + g;
        const float s = inv[mt][hi];
        uint4 o0, o1;  // columns 16 t .. + 7 and 16 t + 8 .. + 15 of this half
        o0.x = pack_bf16x2(acc[mt][0][2 * hi] * s, acc[mt][1][2 * hi] * s);
        o0.y = pack_bf16x2(acc[mt][2][2 * hi] * s, acc[mt][3][2 * hi] * s);
        o0.z = pack_bf16x2(acc[mt][4][2 * hi] * s, acc[mt][5][2 * hi] * s);
        o0.w = pack_bf16x2(acc[mt][6][2 * hi] * s, acc[mt][7][2 * hi] * s);
        o1.x = pack_bf16x2(acc[mt][0][2 * hi + 1] * s, acc[mt][1][2 * hi + 1] * s);
        o1.y = pack_bf16x2(acc[mt][2][2 * hi + 1] * s, acc[mt][3][2 * hi + 1] * s);
        o1.z = pack_bf16x2(acc[mt][4][2 * hi + 1] * s, acc[mt][5][2 * hi + 1] * s);
        o1.w = pack_bf16x2(acc[mt][6][2 * hi + 1] * s, acc[mt][7][2 * hi + 1] * s);
        st_shared_v4(f_addr(tile, row, 8 * h + 2 * t), o0);
        st_shared_v4(f_addr(tile, row, 8 * h + 2 * t + 1), o1);
      }
  }
  __syncwarp();
}

__global__ void __launch_bounds__(kFWarps * 32, 1)
round_fused2_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    const __grid_constant__ CUtensorMap tm_ko, const __grid_constant__ CUtensorMap tm_vo, const FusedArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if ((smem_u32(smem) & 1023u) != 0u) {  // the swizzle pattern needs 1024-byte aligned tiles
    if (threadIdx.x == 0) atomicExch(a.status, 2);
    return;
  }
  const uint32_t tile = smem_u32(smem) + (uint32_t)warp * kFStage;
  unsigned char* extra = smem + (size_t)kFWarps * kFStage + (size_t)warp * kFExtra;
  int* d1 = reinterpret_cast<int*>(extra);        // [64] degrees after round 1, in intermediate order
  int* d2 = reinterpret_cast<int*>(extra + 256);  // [32] degrees after round 2
  const uint32_t bar = smem_u32(extra + 384);

  if (lane == 0) {
    mbar_init(bar, 1);
    mbar_init_fence();
  }
  __syncwarp();

  const int64_t stride = (int64_t)gridDim.x * kFWarps;
  int64_t item = (int64_t)blockIdx.x * kFWarps + warp;
  auto fetch = [&](const CUtensorMap* tm, int64_t it) {
    const uint32_t lh = (uint32_t)it / a.units, u = (uint32_t)it - lh * a.units;
    const int tok = (int)(a.lo + (int64_t)u * kFUnit);
    mbar_arrive_expect_tx(bar, kFStage);
    tma_load_3d(tile, tm, 0, tok, (int)lh, bar);
    tma_load_3d(tile + kFHalf, tm, 64, tok, (int)lh, bar);
  };
  if (item < a.n_items && lane == 0) fetch(&tm_k, item);

  uint32_t parity = 0;
  for (; item < a.n_items; item += stride) {
    const uint32_t lh = (uint32_t)item / a.units, u = (uint32_t)item - lh * a.units;
    const int out_row = (int)(a.lo + (int64_t)u * 32);
    int best_q0 = 0, best_q1 = 0, best_r2 = 0;  // lane i: the B index A token i merges into (round 1 chunk 0 / 1, round 2)
#pragma unroll 1
    for (int ph = 0; ph < 2; ++ph) {  // 0: the K tile (matching and merged keys), 1: the V tile (the same clusters)
      if (!mbar_wait(bar, parity)) {
        if (lane == 0) atomicExch(a.status, 1);
        mbar_wait(bar, parity);  // the copies may still land: one more bounded wait before leaving
        return;
      }
      parity ^= 1;
      __syncwarp();
#pragma unroll 1
      for (int it = 0; it < 3; ++it) {  // round 1 on rows 0-63 and 64-127, then round 2 on the 64 centroids
        const int row0 = it == 1 ? 64 : 0, dst0 = it == 1 ? 32 : 0;
        int best;
        if (ph == 0) {
          best = match64(tile, row0, lane);
          if (it < 2) {
            d1[32 * it + lane] = 1;
            __syncwarp();
            atomicAdd(&d1[32 * it + best], 1);
          } else {
            d2[lane] = d1[2 * lane + 1];
            __syncwarp();
            atomicAdd(&d2[best], d1[2 * lane]);
          }
          __syncwarp();
          if (it == 0) best_q0 = best;
          if (it == 1) best_q1 = best;
          if (it == 2) best_r2 = best;
        } else {
          best = it == 0 ? best_q0 : (it == 1 ? best_q1 : best_r2);
        }
        merge64(tile, row0, dst0, best, it < 2 ? nullptr : d1, it < 2 ? d1 + 32 * it : d2, lane);
      }
      fence_async_smem();  // the TMA store reads the rows through the asynchronous proxy
      __syncwarp();
      if (lane == 0) {
        const CUtensorMap* tmo = ph == 0 ? &tm_ko : &tm_vo;
        tma_store_3d(tmo, 0, out_row, (int)lh, tile);
        tma_store_3d(tmo, 64, out_row, (int)lh, tile + kFHalf);
        bulk_commit();
      }
      if (ph == 0) {
        const int64_t di = (int64_t)lh * a.dst_cap + out_row + lane;
        const int dg = d2[lane];
        a.deg_dst[di] = dg;
        if (a.logdeg_dst) a.logdeg_dst[di] = logf((float)dg);
        if (a.assign1) {
          // round 1: token -> intermediate slot; round 2: intermediate slot -> final slot (composed by the caller)
          const int s1 = (int)(a.lo + (int64_t)u * 64);
          int32_t* as1 = a.assign1 + (int64_t)lh * a.stride1 + a.lo + (int64_t)u * kFUnit;
          as1[2 * lane] = s1 + best_q0;
          as1[2 * lane + 1] = s1 + lane;
          as1[64 + 2 * lane] = s1 + 32 + best_q1;
          as1[64 + 2 * lane + 1] = s1 + 32 + lane;
          int32_t* as2 = a.assign2 + (int64_t)lh * a.stride2 + s1;
          as2[2 * lane] = out_row + best_r2;
          as2[2 * lane + 1] = out_row + lane;
        }
      }
      if (lane == 0) {
        bulk_wait_read();  // the store has read the stage: the next tile may land in it
        fence_async_smem();
        if (ph == 0)
          fetch(&tm_v, item);
        else if (item + stride < a.n_items)
          fetch(&tm_k, item + stride);
      }
      __syncwarp();
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
  if (!make_map(&tm_k, r.k_src, r.src_cap, r.LH, kFUnit, true) || !make_map(&tm_v, r.v_src, r.src_cap, r.LH, kFUnit, true) ||
      !make_map(&tm_ko, r.k_dst, r.dst_cap, r.LH, 32, false) || !make_map(&tm_vo, r.v_dst, r.dst_cap, r.LH, 32, false))
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
  const size_t smem = (size_t)kFWarps * (kFStage + kFExtra);
  cudaError_t e = cudaFuncSetAttribute(round_fused2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return cudaErrorInvalidValue;
  const int64_t ctas = std::min<int64_t>(sms, (a.n_items + kFWarps - 1) / kFWarps);
  round_fused2_kernel<<<(unsigned)ctas, kFWarps * 32, smem, st>>>(tm_k, tm_v, tm_ko, tm_vo, a);
  return cudaGetLastError();
}

}  // namespace ckv
