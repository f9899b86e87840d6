// Chunked Soft Matching round, tile kernel: bf16, head_dim 128, chunk 64 / 128 / 256, every selection mode.
//
// Persistent CTAs walk the chunks of all (layer, head) slabs.  A chunk's K tile and V tile are fetched ahead
// of use with 16-byte asynchronous copies (every thread issues its share) into padded shared-memory rows,
// A tokens first, then B tokens; one commit group per tile.  Per chunk:
//   Sec. 5.2  the A x B dot products on tensor cores (ldmatrix + mma.sync m16n8k16, bf16 in, fp32
//             accumulate); squared key norms from the diagonals of X X^T blocks built from the same
//             fragments; cosine of Eq. 2; row argmax with the lowest B position on ties
//   Sec. 5.3  selection: every edge, the best m of the chunk, or the flags a per-head ranking wrote;
//             or stop after the matching and write the edges for that ranking (then V is never fetched)
//   Eq. 5     the weighted sums over each B token's merged A tokens are one more contraction, W X_A with
//             W[b, a] = n_a if a merges into b else 0 (built in registers, exact in bf16 piece by piece) and
//             X_A the A rows of the K and V tiles, again on tensor cores with fp32 accumulation; all-zero
//             blocks of W are skipped.  The epilogue adds the B token's own term, divides by the summed
//             degree, rounds to bf16 and writes the centroid over the B token's row in the tile; the
//             surviving rows then leave with coalesced 16-byte stores
// Survivors keep their order; a centroid sits at its B token's place.  A shorter last chunk is handled
// in place (rows beyond its length are never copied and never read as candidates).
#include <algorithm>
#include <climits>
#include <cstdint>

#include "ckv_common.cuh"
#include "ckv_internal.h"
#include "ckv_ptx.cuh"

namespace ckv {

namespace {

using namespace ptx;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

constexpr int kTD = 128;          // head_dim
constexpr int kTRowBytes = 256;   // one bf16 row
constexpr int kTStride = 272;     // padded row in shared memory: consecutive rows shift by one 16-byte bank group

template <int C>
struct TileCfg {
  static constexpr int W = (C == 256) ? 16 : 8;  // warps per CTA
  static constexpr int T = W * 32;
  static constexpr int M = C / 2;             // A tokens (rows of the similarity tile) = B tokens (columns)
  static constexpr int MT = C / 32;           // m tiles of 16 A tokens (matching) or 16 B tokens (merge)
  static constexpr int NG = W / MT;           // warps that share an m tile: column groups / column slices
  static constexpr int NTW = (C / 16) / NG;   // matching: n tiles of 8 B tokens per warp
  static constexpr int NTM = 32 / NG;         // merge: n tiles of 8 columns of K | V per warp
  static constexpr int NW = (M + 31) / 32;    // words of the selection mask
  static constexpr int PK = (C == 64) ? 2 : 1;  // the K tile is fetched this many items ahead
  static constexpr int PV = (C == 64) ? 2 : 0;  // the V tile likewise (0: at the start of its own item)
  static constexpr int NK = PK + 1;             // K tiles resident
  static constexpr int NV = PV + 1;             // V tiles resident
  static constexpr int kTile = C * kTStride;
  // offsets
  static constexpr int oK = 0;
  static constexpr int oV = oK + NK * kTile;
  static constexpr int oInv = oV + NV * kTile;       // float [C]  inverse key norms by staged row (B rows only)
  static constexpr int oDeg = oInv + C * 4;          // int   [C]  degrees by local offset
  static constexpr int oBestS = oDeg + C * 4;        // float [M]
  static constexpr int oBestB = oBestS + M * 4;      // int   [M]  B index (0 .. nB-1) or -1
  static constexpr int oPartS = oBestB + M * 4;      // float [M][NG]
  static constexpr int oPartB = oPartS + M * NG * 4; // int   [M][NG]
  static constexpr int oMask = oPartB + M * NG * 4;  // uint  [4]  selection bits by A index
  static constexpr int oBlk = oMask + 16;            // uint  [8]  per m tile of B tokens: which 16-token groups of A merge into it
  static constexpr int oNewDeg = oBlk + 32;          // int   [C]  degree of each output row
  static constexpr int oDsum = oNewDeg + C * 4;      // int   [M]  summed degree of each B token's cluster
  static constexpr int oTw = oDsum + M * 4;          // uint  [3][M]  per A token: target B index << 16 | bf16 weight piece
  static constexpr int oRowOf = oTw + 3 * M * 4;     // ushort[C]  staged row of each output row
  static constexpr int kBytes = oRowOf + C * 2;
  static constexpr int kCtasPerSm = (C == 256) ? 1 : 2;
};

// shared-memory row of local token o: A tokens (even o) in rows [0, C/2), B tokens (odd o) behind them
template <int C>
__device__ __forceinline__ int srow(int o) {
  return ((o & 1) ? C / 2 : 0) + (o >> 1);
}

// selected A tokens with index below x
template <int NW>
__device__ __forceinline__ int sel_below(const uint32_t* mask, int x) {
  int cnt = 0;
#pragma unroll
  for (int w = 0; w < NW; ++w) {
    const int lim = x - 32 * w;
    const uint32_t m = mask[w];
    cnt += lim >= 32 ? __popc(m) : (lim > 0 ? __popc(m & ((1u << lim) - 1u)) : 0);
  }
  return cnt;
}

// Position of a CTA in its walk over the items (chunk `ch` of slab `lh`), advanced without divisions.
struct Cursor {
  int lh, ch;
};

template <int C>
__global__ void __launch_bounds__(TileCfg<C>::T, TileCfg<C>::kCtasPerSm) round_tile_kernel(const RoundArgs a) {
  using Cfg = TileCfg<C>;
  constexpr int T = Cfg::T, W = Cfg::W, M = Cfg::M, MT = Cfg::MT, NG = Cfg::NG, NTW = Cfg::NTW, NTM = Cfg::NTM, NW = Cfg::NW;
  constexpr int NK = Cfg::NK, NV = Cfg::NV, PK = Cfg::PK, PV = Cfg::PV;
  static_assert(PV == PK || PV == 0, "the V tile is fetched together with the K tile or at the start of its own item");
  extern __shared__ __align__(128) unsigned char smem[];
  if (!a.overlap) griddep_wait();  // (an overlap launch waits at its end instead)
  griddep_launch();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int mt = warp % MT, ng = warp / MT;  // this warp's m tile and its column group / slice
  const uint32_t s_base = smem_u32(smem);
  float* inv_nrm = reinterpret_cast<float*>(smem + Cfg::oInv);
  int* degs = reinterpret_cast<int*>(smem + Cfg::oDeg);
  float* best_s = reinterpret_cast<float*>(smem + Cfg::oBestS);
  int* best_b = reinterpret_cast<int*>(smem + Cfg::oBestB);
  float* part_s = reinterpret_cast<float*>(smem + Cfg::oPartS);
  int* part_b = reinterpret_cast<int*>(smem + Cfg::oPartB);
  uint32_t* selmask = reinterpret_cast<uint32_t*>(smem + Cfg::oMask);
  uint32_t* blk = reinterpret_cast<uint32_t*>(smem + Cfg::oBlk);
  int* newdeg = reinterpret_cast<int*>(smem + Cfg::oNewDeg);
  int* dsum = reinterpret_cast<int*>(smem + Cfg::oDsum);
  uint32_t* tw = reinterpret_cast<uint32_t*>(smem + Cfg::oTw);
  unsigned short* row_of = reinterpret_cast<unsigned short*>(smem + Cfg::oRowOf);

  const int mode = a.mode;
  const bool need_sim = mode != kModeExternal;
  const bool need_v = mode != kModeMatchOnly;
  const bool need_cos = mode == kModeMatchOnly || mode == kModeChunkTopM;  // the ranking needs |a| as well
  const __nv_bfloat16* k_src = reinterpret_cast<const __nv_bfloat16*>(a.k_src);
  const __nv_bfloat16* v_src = reinterpret_cast<const __nv_bfloat16*>(a.v_src);
  __nv_bfloat16* k_dst = reinterpret_cast<__nv_bfloat16*>(a.k_dst);
  __nv_bfloat16* v_dst = reinterpret_cast<__nv_bfloat16*>(a.v_dst);
  const int n_chunks = a.n_chunks, LH = a.LH;
  const int n_launch = a.n_launch, ch_end = a.chunk_first + n_launch;  // this launch's chunks of every slab
  const int step_lh = (int)gridDim.x / n_launch, step_ch = (int)gridDim.x % n_launch;
  auto advance = [&](Cursor& c) {
    c.lh += step_lh;
    c.ch += step_ch;
    if (c.ch >= ch_end) {
      c.ch -= n_launch;
      ++c.lh;
    }
  };

  // Rows a shorter chunk leaves unwritten are multiplied by zero weights in the merge: they must hold finite numbers.
  for (uint32_t off = tid * 16u; off < (uint32_t)(NK + NV) * Cfg::kTile; off += T * 16u)
    asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(s_base + off), "r"(0u) : "memory");
  __syncthreads();

  // Fetch the K or V tile of the item at cursor c (the CTA's n-th): every thread copies 16-byte pieces, 16 threads
  // per token row.  Always closes a commit group, also when there is nothing to fetch, so that the counts below hold.
  auto issue = [&](const Cursor& c, int n, bool is_v) {
    if (c.lh < LH && (!is_v || need_v)) {
      const int64_t beg = a.lo + (int64_t)c.ch * C;
      const int clen = (int)min((int64_t)C, a.hi - beg);
      const int buf = n % (is_v ? NV : NK);
      const uint32_t dst = s_base + (is_v ? Cfg::oV : Cfg::oK) + (uint32_t)buf * Cfg::kTile + (uint32_t)(tid & 15) * 16u;
      const __nv_bfloat16* src = (is_v ? v_src : k_src) + ((int64_t)c.lh * a.src_cap + beg) * kTD + (tid & 15) * 8;
#pragma unroll 4
      for (int o = tid >> 4; o < clen; o += T / 16)
        cp_async16(dst + (uint32_t)srow<C>(o) * kTStride, src + (int64_t)o * kTD);
    }
    cp_async_commit();
  };
  // Groups are committed in the order V(n + PV), K(n + PK) at the start of item n, after a prologue of the same shape.
  Cursor cur{(int)blockIdx.x / n_launch, a.chunk_first + (int)blockIdx.x % n_launch};
  Cursor ahead = cur;  // item n + PK
  for (int j = 0; j < PK; ++j) {
    if (PV == PK) issue(ahead, j, true); else cp_async_commit();
    issue(ahead, j, false);
    advance(ahead);
  }

  for (int n = 0; cur.lh < LH; ++n, advance(cur), advance(ahead)) {
    // every thread is past the previous item (barrier at its end): the buffers these copies overwrite are free
    issue(PV == PK ? ahead : cur, n + PV, true);
    issue(ahead, n + PK, false);
    const int64_t lh = cur.lh;
    const int ch = cur.ch;
    const int64_t beg = a.lo + (int64_t)ch * C;
    const int clen = (int)min((int64_t)C, a.hi - beg);
    const int nA = (clen + 1) >> 1, nB = clen >> 1;
    const int64_t eslot = lh * a.edge_stride + (int64_t)ch * M;
    const uint32_t k_s = s_base + Cfg::oK + (uint32_t)(n % NK) * Cfg::kTile;
    const uint32_t v_s = s_base + Cfg::oV + (uint32_t)(n % NV) * Cfg::kTile;

    // loads that are only needed after the matching: issue them now
    int my_deg = 1, ext_b = -1, ext_sel = 0;
    if (a.deg_src && tid < clen) my_deg = a.deg_src[lh * a.src_cap + beg + tid];
    if (mode == kModeExternal && tid < nA) {
      ext_b = a.edge_b[eslot + tid];
      ext_sel = a.sel[eslot + tid];
    }
    const int64_t out_base = (mode == kModeExternal) ? (int64_t)a.chunk_out_off[lh * n_chunks + ch]
                                                     : a.out_lo + (int64_t)ch * a.out_stride;

    cp_async_wait<2 * PK>();  // K(n) was committed 2 PK groups ago
    __syncthreads();          // S0: every thread's pieces of the K tile have landed

    if (tid < clen) {
      degs[tid] = my_deg;
      if (tid & 1) dsum[tid >> 1] = my_deg;  // a cluster starts with its B token's own degree
    }
    if (tid < MT) blk[tid] = 0u;

    float acc[NTW][4];
    float inva[2] = {1.f, 1.f};
    if (need_sim) {
      // ---- dot products: this warp's m tile (16 A tokens) against its NTW n tiles (8 B tokens each);
      //      squared norms from diagonals: of A A^T for the m tile, of B B^T for the n tiles this warp is in charge of
      constexpr bool kPairs = NTW >= 2;
      constexpr int kNormUnits = kPairs ? NTW / 2 : 1;      // pairs of n tiles (or the single n tile) of this column group
      const bool norm_duty = mt < kNormUnits;                // the MT warps of a column group split its units
      const int nu = kPairs ? 2 * mt : 0;                    // first n tile of this warp's unit
      float na0[4] = {0.f, 0.f, 0.f, 0.f}, na1[4] = {0.f, 0.f, 0.f, 0.f};
      float nb0[4] = {0.f, 0.f, 0.f, 0.f}, nb1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < NTW; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
      const uint32_t a_addr = k_s + (uint32_t)(mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * kTStride + (uint32_t)(lane >> 4) * 16u;
      const uint32_t b_addr = k_s + (uint32_t)(M + ng * NTW * 8 + (lane & 7)) * kTStride + (uint32_t)(lane >> 3) * 16u;
#pragma unroll
      for (int kq = 0; kq < 4; ++kq) {
        uint32_t fa0[4], fa1[4];
        ldsm_x4(a_addr + 64u * kq, fa0);        // k = 32 kq .. +15
        ldsm_x4(a_addr + 64u * kq + 32u, fa1);  // k = 32 kq + 16 .. +31
#pragma unroll
        for (int j = 0; j < NTW; ++j) {
          uint32_t fb[4];
          ldsm_x4(b_addr + (uint32_t)j * 8u * kTStride + 64u * kq, fb);
          mma_bf16(acc[j], fa0[0], fa0[1], fa0[2], fa0[3], fb[0], fb[1]);
          mma_bf16(acc[j], fa1[0], fa1[1], fa1[2], fa1[3], fb[2], fb[3]);
        }
        if (need_cos) {  // rows 0-7 of the m tile as columns, then rows 8-15
          mma_bf16(na0, fa0[0], fa0[1], fa0[2], fa0[3], fa0[0], fa0[2]);
          mma_bf16(na0, fa1[0], fa1[1], fa1[2], fa1[3], fa1[0], fa1[2]);
          mma_bf16(na1, fa0[0], fa0[1], fa0[2], fa0[3], fa0[1], fa0[3]);
          mma_bf16(na1, fa1[0], fa1[1], fa1[2], fa1[3], fa1[1], fa1[3]);
        }
        if (norm_duty) {
          uint32_t p[4], q[4] = {0u, 0u, 0u, 0u};
          ldsm_x4(b_addr + (uint32_t)nu * 8u * kTStride + 64u * kq, p);
          if (kPairs) ldsm_x4(b_addr + (uint32_t)(nu + 1) * 8u * kTStride + 64u * kq, q);
          // rows 0-7 <- n tile nu, rows 8-15 <- n tile nu + 1 (zero when there is none); columns: nu, then nu + 1
          mma_bf16(nb0, p[0], q[0], p[1], q[1], p[0], p[1]);
          mma_bf16(nb0, p[2], q[2], p[3], q[3], p[2], p[3]);
          if (kPairs) {
            mma_bf16(nb1, p[0], q[0], p[1], q[1], q[0], q[1]);
            mma_bf16(nb1, p[2], q[2], p[3], q[3], q[2], q[3]);
          }
        }
      }
      // the diagonal entry (row r, column r) of a 16 x 8 block sits in lane 4 r' + r'/2 (r' = r mod 8), register (r' & 1) (+2 for rows 8-15)
      if (norm_duty && t == (g >> 1)) {
        const float s0 = (g & 1) ? nb0[1] : nb0[0];
        inv_nrm[M + (ng * NTW + nu) * 8 + g] = s0 > 0.f ? rsqrtf(s0) : 0.f;  // a zero key has similarity 0 with everything
        if (kPairs) {
          const float s1 = (g & 1) ? nb1[3] : nb1[2];
          inv_nrm[M + (ng * NTW + nu + 1) * 8 + g] = s1 > 0.f ? rsqrtf(s1) : 0.f;
        }
      }
      if (need_cos) {
        const float s0 = (g & 1) ? na0[1] : na0[0], s1 = (g & 1) ? na1[3] : na1[2];
        const float i0 = s0 > 0.f ? rsqrtf(s0) : 0.f, i1 = s1 > 0.f ? rsqrtf(s1) : 0.f;
        const int src_lane = (lane & ~3) | (g >> 1);
        inva[0] = __shfl_sync(0xffffffffu, i0, src_lane);
        inva[1] = __shfl_sync(0xffffffffu, i1, src_lane);
      }
      __syncthreads();  // S1: the B norms are visible

      // ---- Eq. 2 and the row argmax inside this warp's columns
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const int ai = mt * 16 + g + 8 * hi;
        float bv = -INFINITY;
        int bi = INT_MAX;
#pragma unroll
        for (int j = 0; j < NTW; ++j) {
          const int bj0 = (ng * NTW + j) * 8 + 2 * t;
          const float2 invb = *reinterpret_cast<const float2*>(inv_nrm + M + bj0);
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            float s = acc[j][2 * hi + e] * (e ? invb.y : invb.x) * inva[hi];
            s += 0.f;  // -0 -> +0, so that the ranking key orders zeros as equal
            if (bj0 + e < nB && s > bv) {
              bv = s;
              bi = bj0 + e;
            }
          }
        }
#pragma unroll
        for (int o = 1; o <= 2; o <<= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > bv || (ov == bv && oi < bi)) {
            bv = ov;
            bi = oi;
          }
        }
        if (t == 0) {
          part_s[ai * NG + ng] = bv;
          part_b[ai * NG + ng] = bi;
        }
      }
    }
    cp_async_wait<2 * PV + 1>();  // V(n) was committed 2 PV + 1 groups ago
    // S2: the V tile has landed, the partial argmaxes are visible; do the weights need more than one bf16 piece?
    // (the barrier's reduction is a predicate, not a bitwise OR: ask for the third piece only when a second is needed)
    int n_pieces = 1;
    if (__syncthreads_or(my_deg > 255)) n_pieces = __syncthreads_or(my_deg > 65535) ? 3 : 2;

    // ---- one edge per A token
    if (tid < M) {
      float bv = -INFINITY;
      int bi = -1;
      if (need_sim) {
        if (tid < nA && nB > 0) {
#pragma unroll
          for (int q = 0; q < NG; ++q) {  // column groups in increasing column order: strict > keeps the lowest index
            const float ps = part_s[tid * NG + q];
            const int pb = part_b[tid * NG + q];
            if (pb != INT_MAX && (bi < 0 || ps > bv)) {
              bv = ps;
              bi = pb;
            }
          }
        }
        best_s[tid] = bv;
      } else if (tid < nA) {
        bi = ext_b >= 0 ? (ext_b >> 1) : -1;  // stored as the B token's local offset 2 b + 1
      }
      best_b[tid] = bi;
      if (mode == kModeMatchOnly) {
        a.edge_sim[eslot + tid] = bv;
        a.edge_b[eslot + tid] = bi >= 0 ? 2 * bi + 1 : -1;
      }
    }
    if (mode == kModeMatchOnly) {
      __syncthreads();
      continue;
    }

    // ---- Sec. 5.3: which edges are merged
    if (mode == kModeChunkTopM) __syncthreads();  // the ranking reads every edge of the chunk
    if (tid < 32 * NW) {
      int s = 0;
      const int ai = tid;
      if (ai < M) {
        const int bi = best_b[ai];
        if (ai < nA && bi >= 0) {
          if (mode == kModeAll) {
            s = 1;
          } else if (mode == kModeChunkTopM) {
            const int m = (clen == C) ? a.m_full : a.m_tail;
            const float mine = best_s[ai];
            int rank = 0;  // edges of this chunk ranked before mine: higher similarity, or equal and earlier
            for (int o = 0; o < nA; ++o) {
              const float other = best_s[o];
              rank += (other > mine || (other == mine && o < ai)) ? 1 : 0;
            }
            s = rank < m ? 1 : 0;
          } else {
            s = ext_sel ? 1 : 0;
          }
        }
        // the A token's column of W: target B index and its degree as exact bf16 pieces (8 bits each)
        const int da = ai < nA ? degs[2 * ai] : 0;
        const uint32_t tgt = s ? (uint32_t)bi << 16 : 0xffff0000u;
        tw[ai] = tgt | (__float_as_uint((float)(da & 255)) >> 16);
        tw[M + ai] = tgt | (__float_as_uint((float)(da & 0xff00)) >> 16);
        tw[2 * M + ai] = tgt | (__float_as_uint((float)(da & 0xff0000)) >> 16);
        if (s) {
          atomicAdd(&dsum[bi], da);
          atomicOr(&blk[bi >> 4], 1u << (ai >> 4));
        }
      }
      const uint32_t bits = __ballot_sync(0xffffffffu, s != 0);
      if (lane == 0) selmask[warp] = bits;
    }
    __syncthreads();  // S3

    // ---- output order: survivors keep their order, a merged A token shares its B token's slot
    if (tid < clen) {
      const int ai = tid >> 1;
      const bool gone = !(tid & 1) && ((selmask[ai >> 5] >> (ai & 31)) & 1u);
      const int keeper = gone ? 2 * best_b[ai] + 1 : tid;
      const int op = keeper - sel_below<NW>(selmask, (keeper + 1) >> 1);
      if (!gone) {
        row_of[op] = (unsigned short)srow<C>(tid);
        newdeg[op] = (tid & 1) ? dsum[ai] : degs[tid];
      }
      if (a.assign) a.assign[lh * a.assign_stride + beg + tid] = (int32_t)(out_base + op);
    }

    // ---- Eq. 5: acc[b, :] = sum_a W[b, a] X_A[a, :] for this warp's 16 B tokens and its NTM x 8 columns of K | V
    {
      uint32_t todo = blk[mt];  // 16-token groups of A with a member in this m tile
      if (todo) {
        const int b0 = mt * 16 + g, b1 = b0 + 8;
        const uint32_t col = (uint32_t)(ng * NTM * 16) & 255u;                       // byte offset inside the row
        const uint32_t tile = ((ng * NTM * 16) >> 8) ? v_s : k_s;                    // first half of the slices: K, second: V
        const uint32_t x_addr = tile + (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * kTStride + col + (uint32_t)(lane >> 4) * 16u;
        float oacc[NTM][4];
#pragma unroll
        for (int j = 0; j < NTM; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;
        while (todo) {
          const int ks = __ffs(todo) - 1;
          todo &= todo - 1;
          for (int piece = 0; piece < n_pieces; ++piece) {
            const uint32_t* twp = tw + piece * M + 16 * ks + 2 * t;
            const uint2 w01 = *reinterpret_cast<const uint2*>(twp);
            const uint2 w23 = *reinterpret_cast<const uint2*>(twp + 8);
            auto pick = [](uint32_t w, int b) { return (int)(w >> 16) == b ? (w & 0xffffu) : 0u; };
            const uint32_t a0 = pick(w01.x, b0) | (pick(w01.y, b0) << 16);
            const uint32_t a1 = pick(w01.x, b1) | (pick(w01.y, b1) << 16);
            const uint32_t a2 = pick(w23.x, b0) | (pick(w23.y, b0) << 16);
            const uint32_t a3 = pick(w23.x, b1) | (pick(w23.y, b1) << 16);
#pragma unroll
            for (int jp = 0; jp < NTM / 2; ++jp) {
              uint32_t fx[4];
              ldsm_x4_trans(x_addr + (uint32_t)(16 * ks) * kTStride + 32u * jp, fx);
              mma_bf16(oacc[2 * jp], a0, a1, a2, a3, fx[0], fx[1]);
              mma_bf16(oacc[2 * jp + 1], a0, a1, a2, a3, fx[2], fx[3]);
            }
          }
        }
        // epilogue: own term, division by the summed degree, rounding; the centroid replaces the B token's row
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
          const int b = hi ? b1 : b0;
          if (b < nB) {
            const int nb = degs[2 * b + 1], ns = dsum[b];
            if (ns != nb) {  // an untouched row stays bit for bit
              const float wb = (float)nb, inv = 1.0f / (float)ns;
              const uint32_t row = tile + (uint32_t)(M + b) * kTStride + col + t * 4u;
#pragma unroll
              for (int j = 0; j < NTM; ++j) {
                uint32_t x;
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(x) : "r"(row + 16u * j));
                const float o0 = fmaf(wb, __uint_as_float(x << 16), oacc[j][2 * hi]) * inv;
                const float o1 = fmaf(wb, __uint_as_float(x & 0xffff0000u), oacc[j][2 * hi + 1]) * inv;
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(row + 16u * j), "r"(pack_bf16x2(o0, o1)) : "memory");
              }
            }
          }
        }
      }
    }
    __syncthreads();  // S4: the tile rows hold the final values, row_of and newdeg are complete

    // ---- surviving rows leave in order: 16 threads per 256-byte row of K, 16 per row of V
    const int n_out = clen - sel_below<NW>(selmask, M);
    {
      unsigned char* kd = reinterpret_cast<unsigned char*>(k_dst + (lh * a.dst_cap + out_base) * kTD);
      unsigned char* vd = reinterpret_cast<unsigned char*>(v_dst + (lh * a.dst_cap + out_base) * kTD);
      const uint32_t piece = (uint32_t)(tid & 15) * 16u;
      const bool is_v = (tid & 16) != 0;
      const uint32_t tile = is_v ? v_s : k_s;
      unsigned char* dst = (is_v ? vd : kd) + piece;
#pragma unroll 2
      for (int op = tid >> 5; op < n_out; op += W) {
        uint4 x;
        ld_shared_v4(tile + (uint32_t)row_of[op] * kTStride + piece, x);
        *reinterpret_cast<uint4*>(dst + (size_t)op * kTRowBytes) = x;
      }
    }
    if (tid < n_out) {
      const int64_t di = lh * a.dst_cap + out_base + tid;
      const int dg = newdeg[tid];
      a.deg_dst[di] = dg;
      if (a.logdeg_dst) a.logdeg_dst[di] = logf((float)dg);
    }
    __syncthreads();  // S5: the tiles are free
  }
  if (a.overlap) griddep_wait();  // this grid must not complete before the one it ran beside has
}

template <int C>
cudaError_t launch_tile_c(const RoundArgs& a, cudaStream_t st) {
  using Cfg = TileCfg<C>;
  static_assert(Cfg::kBytes <= 227 * 1024, "shared memory");
  const int64_t n_items = (int64_t)a.n_launch * a.LH;
  if (n_items <= 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(round_tile_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kBytes);
  if (e != cudaSuccess) return e;
  const int64_t ctas = std::min<int64_t>((int64_t)sm_count() * Cfg::kCtasPerSm, n_items);
  return launch_dependent(round_tile_kernel<C>, dim3((unsigned)ctas), dim3(Cfg::T), Cfg::kBytes, st, a);
}

}  // namespace

bool round_tile_supported(const RoundArgs& a, int dtype, int D) {
  return dtype == 1 && D == 128 && (a.chunk == 64 || a.chunk == 128 || a.chunk == 256);
}

cudaError_t launch_round_tile(const RoundArgs& a, cudaStream_t st) {
  switch (a.chunk) {
    case 64: return launch_tile_c<64>(a, st);
    case 128: return launch_tile_c<128>(a, st);
    case 256: return launch_tile_c<256>(a, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace ckv
