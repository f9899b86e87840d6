// Chunked Soft Matching round, warp-per-chunk kernel: bf16, chunk 64, head_dim 128, full chunks, every selection mode.
//
// Persistent kernel, one CTA per SM.  Every warp is an independent worker that owns one shared-memory
// stage (a chunk's K tile and V tile, 2 x 16 KiB): it fetches the two tiles with bulk async copies that
// signal the warp's own mbarrier, and while one warp computes, the copies of the others are in flight.
//   Sec. 5.2  the 32 x 32 A x B dot products on tensor cores (mma.sync m16n8k16, bf16 in, fp32
//             accumulate); the squared norms of the B keys come from the same fragments (diagonal of
//             B B^T); row argmax of dot / |b| (dividing a row by |a| > 0 does not change its argmax)
//   Sec. 5.3  which edges merge: all of them (ratio 1, the leanest instantiation), the best m of the chunk
//             (ranked inside the warp with shuffles), or the flags a per-head ranking wrote; or the kernel
//             stops after the matching and writes the edges (cosine of Eq. 2, target) for that ranking,
//             in which case only the K tile is fetched
//   Eq. 5     degree-weighted sums of K and V rows in fp32 from the staged tiles, divided by the
//             summed degree, rounded to bf16, written with coalesced 8-byte stores
// Waits on the mbarrier are bounded: a warp that gives up records it in the status word and leaves.
#include <algorithm>
#include <cstdint>
#include <type_traits>

#include "ckv_common.cuh"
#include "ckv_internal.h"
#include "ckv_ptx.cuh"

namespace ckv {

namespace {

constexpr int kC = 64;            // chunk size
constexpr int kD = 128;           // head_dim
constexpr int kRowBytes = kD * 2; // one bf16 row
constexpr int kTileBytes = kC * kRowBytes;
constexpr int kStageBytes = 2 * kTileBytes;  // K tile then V tile
constexpr int kExtraBytes = 400;             // per warp: degrees [64] int, best [32] int, mbarrier (8 B), pad

using namespace ptx;

__device__ __forceinline__ void unpack4(uint2 u, float (&f)[4]) {
  f[0] = __uint_as_float(u.x << 16);
  f[1] = __uint_as_float(u.x & 0xffff0000u);
  f[2] = __uint_as_float(u.y << 16);
  f[3] = __uint_as_float(u.y & 0xffff0000u);
}

struct FastArgs {
  const __nv_bfloat16* k_src;
  const __nv_bfloat16* v_src;
  const int32_t* deg_src;  // may be null: all ones
  __nv_bfloat16* k_dst;
  __nv_bfloat16* v_dst;
  int32_t* deg_dst;
  float* logdeg_dst;  // may be null
  int32_t* assign;    // may be null
  int64_t assign_stride;
  int64_t src_cap, dst_cap;
  int64_t lo;       // first token of the middle region in src
  int64_t out_lo;   // where the first chunk's survivors go in dst
  int64_t n_full;   // full chunks per (layer, head)
  int64_t n_items;  // n_full * LH
  int32_t* status;  // device word: set to 1 if a wait gave up
  // selection (unused when every edge merges)
  int32_t mode;            // RoundMode
  int32_t m_full;          // kModeChunkTopM: merges per chunk
  int32_t out_stride;      // survivors of a chunk (kModeAll, kModeChunkTopM)
  int32_t n_chunks;        // chunks per slab: stride of chunk_out_off
  int64_t edge_stride;     // edges per slab: stride of edge_sim, edge_b, sel
  float* edge_sim;         // kModeMatchOnly writes
  int32_t* edge_b;         // kModeMatchOnly writes, kModeExternal reads: local offset of the edge's B token
  const uint8_t* sel;      // kModeExternal: 1 = merge this edge
  const int32_t* chunk_out_off;  // kModeExternal: dst position of the chunk's first survivor
};

enum FastKind : int { kFastAll = 0, kFastSelect = 1, kFastMatch = 2 };

// row of token `pos` of KV head h in a pool's [n_pages, H, page_tokens] grid
__device__ __forceinline__ int64_t page_row(const int32_t* table, int H, int shift, int h, int64_t pos) {
  return (((int64_t)table[pos >> shift] * H + h) << shift) + (pos & (((int64_t)1 << shift) - 1));
}

__device__ __forceinline__ unsigned char* pg_k(const PagedArgs& pg, int l) { return pg.k[l]; }
__device__ __forceinline__ unsigned char* pg_v(const PagedArgs& pg, int l) { return pg.v[l]; }
__device__ __forceinline__ int32_t* pg_deg(const PagedArgs& pg, int l) { return pg.deg[l]; }
__device__ __forceinline__ float* pg_logdeg(const PagedArgs& pg, int l) { return pg.logdeg[l]; }
__device__ __forceinline__ unsigned char* pg_k(const NoPages&, int) { return nullptr; }
__device__ __forceinline__ unsigned char* pg_v(const NoPages&, int) { return nullptr; }
__device__ __forceinline__ int32_t* pg_deg(const NoPages&, int) { return nullptr; }
__device__ __forceinline__ float* pg_logdeg(const NoPages&, int) { return nullptr; }

template <int NW, bool HAS_DEG, int KIND, bool PAGED>
__global__ void __launch_bounds__(NW * 32, 1)
round_fast_kernel(const FastArgs a, const __grid_constant__ typename std::conditional<PAGED, PagedArgs, NoPages>::type pg) {
  extern __shared__ __align__(128) unsigned char smem[];
  griddep_wait();    // ordered launch: everything ahead in the stream has completed
  griddep_launch();  // the next launch may become resident as this grid's CTAs leave
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  constexpr int kStage = KIND == kFastMatch ? kTileBytes : kStageBytes;  // the matching alone stages no V tile
  unsigned char* stage = smem + (size_t)warp * kStage;
  unsigned char* extra = smem + (size_t)NW * kStage + (size_t)warp * kExtraBytes;
  int* degs = reinterpret_cast<int*>(extra);             // [64]
  const uint32_t bar = smem_u32(extra + 384);
  const uint32_t k_s = smem_u32(stage), v_s = k_s + kTileBytes;
  const uint32_t n_full = (uint32_t)a.n_full;
  const bool external = KIND == kFastSelect && a.mode == kModeExternal;  // edges and flags come from global memory

  if (lane == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  const int64_t stride = (int64_t)gridDim.x * NW;
  int64_t item = (int64_t)blockIdx.x * NW + warp;
  auto issue = [&](int64_t it) {
    const uint32_t lh = (uint32_t)it / n_full, ch = (uint32_t)it - lh * n_full;
    mbar_arrive_expect_tx(bar, KIND == kFastMatch ? kTileBytes : kStageBytes);
    if constexpr (PAGED) {
      // a chunk is one run of rows inside a page, or two runs when it straddles a page boundary
      const int l = (int)(lh / (uint32_t)pg.H), h = (int)(lh - (uint32_t)l * pg.H);
      const int64_t pos0 = a.lo + (int64_t)ch * kC, page_tokens = (int64_t)1 << pg.shift;
      const int n1 = (int)min((int64_t)kC, page_tokens - (pos0 & (page_tokens - 1)));
      const int64_t r1 = page_row(pg.src_table, pg.H, pg.shift, h, pos0);
      bulk_load(k_s, pg.k[l] + r1 * kRowBytes, (uint32_t)n1 * kRowBytes, bar);
      if (KIND != kFastMatch) bulk_load(v_s, pg.v[l] + r1 * kRowBytes, (uint32_t)n1 * kRowBytes, bar);
      if (n1 < kC) {
        const int64_t r2 = page_row(pg.src_table, pg.H, pg.shift, h, pos0 + n1);
        bulk_load(k_s + n1 * kRowBytes, pg.k[l] + r2 * kRowBytes, (uint32_t)(kC - n1) * kRowBytes, bar);
        if (KIND != kFastMatch) bulk_load(v_s + n1 * kRowBytes, pg.v[l] + r2 * kRowBytes, (uint32_t)(kC - n1) * kRowBytes, bar);
      }
    } else {
      const int64_t row0 = (int64_t)lh * a.src_cap + a.lo + (int64_t)ch * kC;
      bulk_load(k_s, a.k_src + row0 * kD, kTileBytes, bar);
      if (KIND != kFastMatch) bulk_load(v_s, a.v_src + row0 * kD, kTileBytes, bar);  // the matching alone never reads V
    }
  };
  if (item < a.n_items && lane == 0) issue(item);

  uint32_t parity = 0;
  for (; item < a.n_items; item += stride, parity ^= 1) {
    const uint32_t lh = (uint32_t)item / n_full, ch = (uint32_t)item - lh * n_full;
    const int64_t src_row0 = (int64_t)lh * a.src_cap + a.lo + (int64_t)ch * kC;
    const int64_t eslot = (int64_t)lh * a.edge_stride + (int64_t)ch * (kC / 2);
    int64_t out_row0 = (int64_t)lh * a.dst_cap;
    int ext_b = 1, ext_sel = 0;
    int64_t out_pos0;  // position in the sequence of the chunk's first output row
    if (external) {
      out_pos0 = a.chunk_out_off[(int64_t)lh * a.n_chunks + ch];
      ext_b = a.edge_b[eslot + lane];
      ext_sel = a.sel[eslot + lane];
    } else {
      out_pos0 = a.out_lo + (int64_t)ch * a.out_stride;
    }
    out_row0 += out_pos0;
    // paged: the layer and head of this slab, and the (at most two) destination pages the chunk's output rows reach
    int pl = 0, ph = 0;
    // output row `op` sits at pool row out_pos0 + op + pg_add0 while it is in the first page (op < pg_first), + pg_add1 behind
    int64_t pg_add0 = 0, pg_add1 = 0;
    int pg_first = 0;
    if constexpr (PAGED) {
      pl = (int)(lh / (uint32_t)pg.H);
      ph = (int)(lh - (uint32_t)pl * pg.H);
      if (KIND != kFastMatch) {
        const int64_t dst_pg0 = out_pos0 >> pg.shift;
        const int64_t dst_id0 = pg.dst_table[min(dst_pg0, pg.dst_last_page)];
        const int64_t dst_id1 = pg.dst_table[min((out_pos0 + kC - 1) >> pg.shift, pg.dst_last_page)];
        pg_first = (int)(((dst_pg0 + 1) << pg.shift) - out_pos0);
        pg_add0 = ((dst_id0 * pg.H + ph) << pg.shift) - (dst_pg0 << pg.shift);
        pg_add1 = ((dst_id1 * pg.H + ph) << pg.shift) - ((dst_pg0 + 1) << pg.shift);
      }
    }
    // row of output row `op` of this chunk: in the destination slab array, or in the destination pool's page grid
    auto dst_row = [&](int op) -> int64_t {
      if constexpr (PAGED) {
        return out_pos0 + op + (op < pg_first ? pg_add0 : pg_add1);
      } else {
        return out_row0 + op;
      }
    };
    if (HAS_DEG && KIND != kFastMatch) {
      if constexpr (PAGED) {
        const int64_t pos0 = a.lo + (int64_t)ch * kC;
        degs[lane] = pg.deg[pl][page_row(pg.src_table, pg.H, pg.shift, ph, pos0 + lane)];
        degs[lane + 32] = pg.deg[pl][page_row(pg.src_table, pg.H, pg.shift, ph, pos0 + lane + 32)];
      } else {
        degs[lane] = a.deg_src[src_row0 + lane];
        degs[lane + 32] = a.deg_src[src_row0 + lane + 32];
      }
    }
    if (!mbar_wait(bar, parity)) {
      if (lane == 0) atomicExch(a.status, 1);
      mbar_wait(bar, parity);  // the copies may still land: give them one more bounded wait before leaving
      return;
    }
    __syncwarp();

    int my_best = ext_b >> 1;  // B index (0..31) chosen by A token `lane`
    float my_s = 0.f;          // its cosine similarity (ranking modes only)
    if (!external) {
      // ---- A x B dot products and the squared norms on tensor cores
      float acc[2][4][4];   // [m tile][n tile][c]: A token 16*mt + g (+8), B index 8*nt + 2t (+1)
      float nacc[2][2][4];  // B B^T diagonals: [pair of n tiles][which of the pair as column operand][c]
      float aacc[2][2][4];  // A A^T diagonals: [m tile][rows 0-7 / 8-15 as column operand][c]
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
          for (int c = 0; c < 4; ++c) nacc[i][j][c] = aacc[i][j][c] = 0.f;

#pragma unroll
      for (int kp = 0; kp < 4; ++kp) {
        // each lane reads 16 contiguous bytes of a row: elements 32*kp + 8*t .. +7.  The same permutation of the
        // contraction index is applied to both operands, so the dot products are unchanged.
        uint4 ra[2][2], rb[4];
        const uint32_t col = 64u * kp + 16u * t;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int hi = 0; hi < 2; ++hi) {
            const uint32_t tok = 2u * (16u * mt + 8u * hi + g);
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(ra[mt][hi].x), "=r"(ra[mt][hi].y), "=r"(ra[mt][hi].z), "=r"(ra[mt][hi].w)
                         : "r"(k_s + tok * kRowBytes + col));
          }
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          const uint32_t tok = 2u * (8u * nt + g) + 1u;
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(rb[nt].x), "=r"(rb[nt].y), "=r"(rb[nt].z), "=r"(rb[nt].w)
                       : "r"(k_s + tok * kRowBytes + col));
        }
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
            if (KIND != kFastAll) {  // the ranking needs |a| too: A A^T with rows 0-7, then rows 8-15, as the column operand
              mma_bf16(aacc[mt][0], a0, a1, a2, a3, a0, a2);
              mma_bf16(aacc[mt][1], a0, a1, a2, a3, a1, a3);
            }
          }
          // B B^T on pairs of n tiles: rows = B indices 16p + g (+8), the diagonal holds the squared norms
#pragma unroll
          for (int p = 0; p < 2; ++p) {
            mma_bf16(nacc[p][0], b0[2 * p], b0[2 * p + 1], b1[2 * p], b1[2 * p + 1], b0[2 * p], b1[2 * p]);
            mma_bf16(nacc[p][1], b0[2 * p], b0[2 * p + 1], b1[2 * p], b1[2 * p + 1], b0[2 * p + 1], b1[2 * p + 1]);
          }
        }
      }

      // squared norm of B index 8*nt + g sits on the diagonal: lane (g, t = g / 2), register g & 1 (+2 for odd nt)
      float inv0[4], inv1[4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const int p = nt >> 1, h = nt & 1;
        const float ss = (g & 1) ? nacc[p][h][2 * h + 1] : nacc[p][h][2 * h];
        const float inv = ss > 0.f ? rsqrtf(ss) : 0.f;
        inv0[nt] = __shfl_sync(0xffffffffu, inv, 9 * t);      // B index 8*nt + 2t     lives in lane 4*(2t) + t
        inv1[nt] = __shfl_sync(0xffffffffu, inv, 9 * t + 4);  // B index 8*nt + 2t + 1 lives in lane 4*(2t+1) + t
      }

      // ---- row argmax (lowest B index on ties); every lane of a quad ends up with the rows of its g
      float row_s[2][2];
      int row_b[2][2];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
          float inva = 1.f;  // dividing a row by |a| > 0 does not change its argmax: only the ranking modes pay for it
          if (KIND != kFastAll) {
            const float ss = (g & 1) ? aacc[mt][hi][2 * hi + 1] : aacc[mt][hi][2 * hi];
            inva = __shfl_sync(0xffffffffu, ss > 0.f ? rsqrtf(ss) : 0.f, (lane & ~3) | (g >> 1));
          }
          float bv = -INFINITY;
          int bi = 0x7fffffff;
#pragma unroll
          for (int nt = 0; nt < 4; ++nt) {
            float s0 = acc[mt][nt][2 * hi] * inv0[nt] * inva + 0.f, s1 = acc[mt][nt][2 * hi + 1] * inv1[nt] * inva + 0.f;
            if (s0 > bv) { bv = s0; bi = 8 * nt + 2 * t; }
            if (s1 > bv) { bv = s1; bi = 8 * nt + 2 * t + 1; }
          }
#pragma unroll
          for (int o = 1; o <= 2; o <<= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          row_s[mt][hi] = bv;
          row_b[mt][hi] = bi;
        }
      // lane = A index i takes row i = 16 mt + 8 hi + g from the quad of g = i & 7
      {
        const int src = 4 * (lane & 7), which = lane >> 3;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int hi = 0; hi < 2; ++hi) {
            const int vb = __shfl_sync(0xffffffffu, row_b[mt][hi], src);
            if (which == 2 * mt + hi) my_best = vb;
            if (KIND != kFastAll) {
              const float vs = __shfl_sync(0xffffffffu, row_s[mt][hi], src);
              if (which == 2 * mt + hi) my_s = vs;
            }
          }
      }
    }

    if (KIND == kFastMatch) {
      a.edge_sim[eslot + lane] = my_s;
      a.edge_b[eslot + lane] = 2 * my_best + 1;
    } else {
      // ---- Sec. 5.3: which edges merge
      unsigned selm = 0xffffffffu;
      if (KIND == kFastSelect) {
        bool s;
        if (external) {
          s = ext_sel != 0;
        } else {
          int rank = 0;  // edges of this chunk ranked before mine: higher similarity, or equal and earlier
#pragma unroll 8
          for (int o = 0; o < 32; ++o) {
            const float other = __shfl_sync(0xffffffffu, my_s, o);
            rank += (other > my_s || (other == my_s && o < lane)) ? 1 : 0;
          }
          s = rank < a.m_full;
        }
        selm = __ballot_sync(0xffffffffu, s);
      }
      auto slot_a = [selm](int i) { return 2 * i - __popc(selm & ((1u << i) - 1u)); };              // A token i, if it survives
      auto slot_b = [selm](int j) { return 2 * j + 1 - __popc(selm & (0xffffffffu >> (31 - j))); };  // B token j

      // ---- Eq. 5: one output row per B token, members gathered from the staged tiles; unmerged A tokens pass through
      int deg_lo = 0, deg_hi = 0;  // degrees of output rows `lane` and `lane + 32`
      __nv_bfloat16* const kbase = (PAGED ? reinterpret_cast<__nv_bfloat16*>(pg_k(pg, pl)) : a.k_dst) + lane * 4;
      __nv_bfloat16* const vbase = (PAGED ? reinterpret_cast<__nv_bfloat16*>(pg_v(pg, pl)) : a.v_dst) + lane * 4;
#pragma unroll 2
      for (int j = 0; j < 32; ++j) {
        if (KIND == kFastSelect && !((selm >> j) & 1u)) {
          const int op = slot_a(j);
          const uint32_t arow = (2u * j) * kRowBytes + lane * 8u;
          uint2 ck, cv;
          asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(ck.x), "=r"(ck.y) : "r"(k_s + arow));
          asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(cv.x), "=r"(cv.y) : "r"(v_s + arow));
          const int64_t orow = dst_row(op);
          *reinterpret_cast<uint2*>(kbase + orow * kD) = ck;
          *reinterpret_cast<uint2*>(vbase + orow * kD) = cv;
          const int n_a = HAS_DEG ? degs[2 * j] : 1;
          if (lane == (op & 31)) (op < 32 ? deg_lo : deg_hi) = n_a;
        }
        unsigned members = __ballot_sync(0xffffffffu, my_best == j && ((selm >> lane) & 1u));
        const int op = KIND == kFastAll ? j : slot_b(j);
        const uint32_t brow = (2u * j + 1u) * kRowBytes + lane * 8u;
        uint2 uk, uv;
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(uk.x), "=r"(uk.y) : "r"(k_s + brow));
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(uv.x), "=r"(uv.y) : "r"(v_s + brow));
        int n_new = HAS_DEG ? degs[2 * j + 1] : 1;
        if (members) {
          float fk[4], fv[4];
          unpack4(uk, fk);
          unpack4(uv, fv);
          if (HAS_DEG) {
            const float wb = (float)n_new;
#pragma unroll
            for (int e = 0; e < 4; ++e) { fk[e] *= wb; fv[e] *= wb; }
          }
          while (members) {
            const int ai = __ffs(members) - 1;
            members &= members - 1;
            const uint32_t arow = (2u * ai) * kRowBytes + lane * 8u;
            uint2 mk, mv;
            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(mk.x), "=r"(mk.y) : "r"(k_s + arow));
            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(mv.x), "=r"(mv.y) : "r"(v_s + arow));
            float gk[4], gv[4];
            unpack4(mk, gk);
            unpack4(mv, gv);
            if (HAS_DEG) {
              const int wa = degs[2 * ai];
              const float w = (float)wa;
              n_new += wa;
#pragma unroll
              for (int e = 0; e < 4; ++e) { fk[e] = fmaf(w, gk[e], fk[e]); fv[e] = fmaf(w, gv[e], fv[e]); }
            } else {
              n_new += 1;
#pragma unroll
              for (int e = 0; e < 4; ++e) { fk[e] += gk[e]; fv[e] += gv[e]; }
            }
          }
          const float inv = 1.0f / (float)n_new;
          uk.x = pack_bf16x2(fk[0] * inv, fk[1] * inv);
          uk.y = pack_bf16x2(fk[2] * inv, fk[3] * inv);
          uv.x = pack_bf16x2(fv[0] * inv, fv[1] * inv);
          uv.y = pack_bf16x2(fv[2] * inv, fv[3] * inv);
        }
        const int64_t orow = dst_row(op);
        *reinterpret_cast<uint2*>(kbase + orow * kD) = uk;  // a B token nobody chose is copied bit for bit
        *reinterpret_cast<uint2*>(vbase + orow * kD) = uv;
        if (lane == (op & 31)) (op < 32 ? deg_lo : deg_hi) = n_new;
      }
      const int n_out = kC - __popc(selm);
      int32_t* const deg_out = PAGED ? pg_deg(pg, pl) : a.deg_dst;
      float* const logdeg_out = PAGED ? pg_logdeg(pg, pl) : a.logdeg_dst;
      if (lane < n_out) {
        const int64_t orow = dst_row(lane);
        deg_out[orow] = deg_lo;
        if (logdeg_out) logdeg_out[orow] = logf((float)deg_lo);
      }
      if (KIND == kFastSelect && lane + 32 < n_out) {
        const int64_t orow = dst_row(lane + 32);
        deg_out[orow] = deg_hi;
        if (logdeg_out) logdeg_out[orow] = logf((float)deg_hi);
      }
      if (a.assign) {
        int32_t* as = a.assign + (int64_t)lh * a.assign_stride + a.lo + (int64_t)ch * kC;
        const int32_t slot0 = (int32_t)out_pos0;
        const bool merged = (selm >> lane) & 1u;
        as[2 * lane] = slot0 + (merged ? slot_b(my_best) : slot_a(lane));  // a merged A token joins its B token's slot
        as[2 * lane + 1] = slot0 + slot_b(lane);
      }
    }

    // ---- this stage is free again: fetch the warp's next chunk
    __syncwarp();
    if (item + stride < a.n_items && lane == 0) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      issue(item + stride);
    }
  }
}

template <int NW, bool HAS_DEG, int KIND, bool PAGED, typename PG>
cudaError_t launch_fast_inst(const FastArgs& a, const PG& pg, cudaStream_t st) {
  const size_t smem = (size_t)NW * ((KIND == kFastMatch ? kTileBytes : kStageBytes) + kExtraBytes);
  const int64_t ctas = std::min<int64_t>(sm_count(), (a.n_items + NW - 1) / NW);
  cudaError_t e = cudaFuncSetAttribute(round_fast_kernel<NW, HAS_DEG, KIND, PAGED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_dependent(round_fast_kernel<NW, HAS_DEG, KIND, PAGED>, dim3((unsigned)ctas), dim3(NW * 32), smem, st, a, pg);
}

template <int NW, int KIND, bool PAGED, typename PG>
cudaError_t launch_fast_kind(const FastArgs& a, const PG& pg, cudaStream_t st) {
  // the matching alone never reads degrees
  return (a.deg_src && KIND != kFastMatch) ? launch_fast_inst<NW, true, KIND, PAGED>(a, pg, st)
                                           : launch_fast_inst<NW, false, KIND, PAGED>(a, pg, st);
}

template <bool PAGED, typename PG>
cudaError_t launch_fast_any(const RoundArgs& r, const PG& pg, int64_t n_full, cudaStream_t st) {
  // r.chunk_first > 0: only the full chunks from that one on (modes whose output offsets are a multiple of the chunk index)
  const int64_t first = r.chunk_first;
  n_full -= first;
  if (n_full <= 0) return cudaSuccess;
  if (first > 0 && r.mode != kModeAll && r.mode != kModeChunkTopM) return cudaErrorInvalidValue;
  FastArgs a{};
  a.k_src = static_cast<const __nv_bfloat16*>(r.k_src);
  a.v_src = static_cast<const __nv_bfloat16*>(r.v_src);
  a.deg_src = r.deg_src;
  a.k_dst = static_cast<__nv_bfloat16*>(r.k_dst);
  a.v_dst = static_cast<__nv_bfloat16*>(r.v_dst);
  a.deg_dst = r.deg_dst;
  a.logdeg_dst = r.logdeg_dst;
  a.assign = r.assign;
  a.assign_stride = r.assign_stride;
  a.src_cap = r.src_cap;
  a.dst_cap = r.dst_cap;
  a.lo = r.lo + first * kC;
  a.out_lo = r.out_lo + first * r.out_stride;
  a.n_full = n_full;
  a.n_items = n_full * r.LH;
  a.status = r.status;
  a.mode = r.mode;
  a.m_full = r.m_full;
  a.out_stride = (int32_t)r.out_stride;
  a.n_chunks = r.n_chunks;
  a.edge_stride = r.edge_stride;
  a.edge_sim = r.edge_sim;
  a.edge_b = r.edge_b;
  a.sel = r.sel;
  a.chunk_out_off = r.chunk_out_off;
  switch (r.mode) {
    case kModeAll: return launch_fast_kind<7, kFastAll, PAGED>(a, pg, st);
    case kModeMatchOnly: return launch_fast_kind<13, kFastMatch, PAGED>(a, pg, st);  // half the bytes per warp: twice the warps
    default: return launch_fast_kind<7, kFastSelect, PAGED>(a, pg, st);
  }
}

}  // namespace

bool round_fast_supported(const RoundArgs& a, int dtype, int D) {
  return dtype == 1 && D == 128 && a.chunk == kC && a.status != nullptr && (int64_t)a.LH * a.n_chunks < (1ll << 31);
}

// The full chunks of a round in any mode.  The shorter last chunk, if any, is left to the tile kernel.
cudaError_t launch_round_fast(const RoundArgs& r, int64_t n_full, cudaStream_t st) { return launch_fast_any<false>(r, NoPages{}, n_full, st); }

cudaError_t launch_round_fast_paged(const RoundArgs& r, const PagedArgs& pg, int64_t n_full, cudaStream_t st) {
  return launch_fast_any<true>(r, pg, n_full, st);
}

}  // namespace ckv
