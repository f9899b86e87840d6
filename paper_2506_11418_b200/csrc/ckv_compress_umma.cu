// Chunked Soft Matching round at chunk 256 (the paper's default), bf16, head_dim 128, full chunks, every selection
// mode: the two contractions of a chunk run on the 5th-generation tensor cores with accumulators in tensor memory.
//
// One persistent CTA (16 warps) per SM walks the chunks.  Per chunk:
//   fetch     the K tile and the V tile arrive by TMA (cp.async.bulk.tensor, 128-byte swizzle); the tensor map views
//             the cache as (column, parity, token pair, slab), so the A tokens (1st, 3rd, ...) and the B tokens land
//             de-interleaved, each as two 128 x 64 operand tiles in the canonical swizzled layout.  K is fetched one
//             chunk ahead
//   Sec. 5.2  S = A B^T, 128 x 128 x 128, eight tcgen05.mma issued by one thread into tensor memory; the inverse key
//             norms come from X X^T diagonals (warp-level mma on the same swizzled tiles); every thread then reads
//             one A token's row of S (tcgen05.ld), scales it to the cosine of Eq. 2 and takes the argmax
//   Sec. 5.3  selection as in the other kernels: every edge, the best m of the chunk, or flags from global memory;
//             or stop after the matching and write the edges
//   Eq. 5     the weighted sums are W X_A with W[b, a] = n_a if a merges into b (written into a swizzled 128 x 64
//             operand tile, 8-bit pieces of the degree are exact in bf16) and X_A the A rows of the K and V tiles as
//             the MN-major operand: tcgen05.mma into 2 x 128 columns of tensor memory.  The epilogue (one thread per
//             centroid row and tile) adds the own term, divides, rounds and overwrites the B row in the tile; with
//             every edge merged the 128 centroid rows are one contiguous tile and leave by TMA store
// mbarrier waits are bounded; if one gives up the CTA records it in the status word, frees its tensor memory and leaves.
#include <cuda.h>

#include <algorithm>
#include <climits>
#include <cstdint>

#include "ckv_common.cuh"
#include "ckv_internal.h"
#include "ckv_ptx.cuh"

namespace ckv {

namespace {

using namespace ptx;

constexpr int kUC = 256;               // chunk
constexpr int kUM = 128;               // A tokens = B tokens per chunk
constexpr int kUD = 128;               // head_dim
constexpr int kUThreads = 512;
constexpr int kHalf = kUM * 128;       // one operand tile: 128 rows x 64 columns (128 bytes), swizzled: 16 KiB
constexpr int kTileU = 4 * kHalf;      // A cols 0-63 | A cols 64-127 | B cols 0-63 | B cols 64-127
constexpr uint32_t kTmemCols = 512;    // S: columns [0, 128); merged K: [128, 256); merged V: [256, 384)

// shared-memory layout (from a 1024-byte aligned base)
constexpr int oUK = 0;                          // two K tiles
constexpr int oUV = 2 * kTileU;                 // one V tile
constexpr int oUW = 3 * kTileU;                 // W operand tile, 128 x 64
constexpr int oUInv = oUW + kHalf;              // float [256] inverse norms: A tokens [0,128), B tokens [128,256)
constexpr int oUDeg = oUInv + 1024;             // int   [256] degrees by local offset
constexpr int oUDsum = oUDeg + 1024;            // int   [128] summed degree of each B token's cluster
constexpr int oUBestB = oUDsum + 512;           // int   [128]
constexpr int oUBestS = oUBestB + 512;          // float [128]
constexpr int oUPartS = oUBestS + 512;          // float [128][4]
constexpr int oUPartB = oUPartS + 2048;         // int   [128][4]
constexpr int oUTw = oUPartB + 2048;            // uint  [3][128]: target B index << 16 | bf16 weight piece
constexpr int oUMask = oUTw + 1536;             // uint  [4]
constexpr int oUNewDeg = oUMask + 16;           // int   [256]
constexpr int oURowOf = oUNewDeg + 1024;        // ushort[256]: (part << 7 | row) of each output row
constexpr int oUBar = oURowOf + 512;            // mbarriers: kfull[2], vfull, sim, merge
constexpr int oUTmem = oUBar + 64;              // tensor-memory base address
constexpr int kUBytes = oUTmem + 16;
constexpr int kUAlign = 1024;

struct UmmaArgs {
  RoundArgs r;
  int64_t n_full;  // full chunks per slab handled here
};

// byte offset of element column `col` (0..127) of row `row` inside a part (A or B) of a swizzled tile
__device__ __forceinline__ uint32_t sw_off(int row, int chunk16 /* 0..15: 16-byte piece of the 256-byte row */) {
  return (uint32_t)(chunk16 >> 3) * kHalf + (uint32_t)row * 128u + (uint32_t)(((chunk16 & 7) ^ (row & 7)) << 4);
}

// instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128; b_mn: the B operand is MN-major
__host__ __device__ constexpr uint32_t umma_idesc(bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn ? 1u : 0u) << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

__global__ void __launch_bounds__(kUThreads, 1)
round_umma_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const __grid_constant__ CUtensorMap tm_ko, const __grid_constant__ CUtensorMap tm_vo, const RoundArgs a,
                  const int n_full) {
  extern __shared__ unsigned char smem_raw[];
  // the operand tiles need 1024-byte alignment (the swizzle pattern repeats every 8 rows of 128 bytes)
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + kUAlign - 1) & ~(uintptr_t)(kUAlign - 1));
  const uint32_t s_base = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  float* inv_nrm = reinterpret_cast<float*>(smem + oUInv);
  int* degs = reinterpret_cast<int*>(smem + oUDeg);
  int* dsum = reinterpret_cast<int*>(smem + oUDsum);
  int* best_b = reinterpret_cast<int*>(smem + oUBestB);
  float* best_s = reinterpret_cast<float*>(smem + oUBestS);
  float* part_s = reinterpret_cast<float*>(smem + oUPartS);
  int* part_b = reinterpret_cast<int*>(smem + oUPartB);
  uint32_t* tw = reinterpret_cast<uint32_t*>(smem + oUTw);
  uint32_t* selmask = reinterpret_cast<uint32_t*>(smem + oUMask);
  int* newdeg = reinterpret_cast<int*>(smem + oUNewDeg);
  unsigned short* row_of = reinterpret_cast<unsigned short*>(smem + oURowOf);
  const uint32_t bar_k[2] = {s_base + oUBar, s_base + oUBar + 8};
  const uint32_t bar_v = s_base + oUBar + 16, bar_sim = s_base + oUBar + 24, bar_mrg = s_base + oUBar + 32;
  const uint32_t w_s = s_base + oUW, v_s = s_base + oUV;

  const int mode = a.mode;
  const bool need_sim = mode != kModeExternal;
  const bool need_v = mode != kModeMatchOnly;
  const bool need_cos = mode == kModeMatchOnly || mode == kModeChunkTopM;
  const int LH = a.LH;
  const int step_lh = (int)gridDim.x / n_full, step_ch = (int)gridDim.x % n_full;
  struct Cur { int lh, ch; };
  auto advance = [&](Cur& c) {
    c.lh += step_lh;
    c.ch += step_ch;
    if (c.ch >= n_full) {
      c.ch -= n_full;
      ++c.lh;
    }
  };

  if (tid == 0) {
    mbar_init(bar_k[0], 1);
    mbar_init(bar_k[1], 1);
    mbar_init(bar_v, 1);
    mbar_init(bar_sim, 1);
    mbar_init(bar_mrg, 1);
    mbar_init_fence();
  }
  if (warp == 0) tmem_alloc(s_base + oUTmem, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + oUTmem);

  // one thread fetches a tile: A tokens (parity 0) and B tokens (parity 1), two 64-column halves each
  auto fetch = [&](const CUtensorMap* tm, uint32_t dst, uint32_t bar, const Cur& c) {
    mbar_arrive_expect_tx(bar, kTileU);
    tma_load_4d(dst, tm, 0, 0, c.ch * kUM, c.lh, bar);
    tma_load_4d(dst + kHalf, tm, 64, 0, c.ch * kUM, c.lh, bar);
    tma_load_4d(dst + 2 * kHalf, tm, 0, 1, c.ch * kUM, c.lh, bar);
    tma_load_4d(dst + 3 * kHalf, tm, 64, 1, c.ch * kUM, c.lh, bar);
  };
  // leave after a wait gave up: the status word is set, tensor memory is returned
  auto bail = [&](uint32_t bar, uint32_t parity) {
    if (tid == 0) atomicExch(a.status, 1);
    mbar_wait(bar, parity);  // copies or MMAs may still complete: one more bounded wait
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
  };

  Cur cur{(int)blockIdx.x / n_full, (int)blockIdx.x % n_full};
  if (tid == 0 && cur.lh < LH) fetch(&tm_k, s_base + oUK, bar_k[0], cur);
  uint32_t ph_v = 0, ph_sim = 0, ph_mrg = 0;

  for (int n = 0; cur.lh < LH; ++n) {
    const int s = n & 1;
    const uint32_t k_s = s_base + oUK + (uint32_t)s * kTileU;
    Cur nxt = cur;
    advance(nxt);
    if (tid == 0) {
      bulk_wait_read();  // the stores of the previous chunk have read their tiles
      if (nxt.lh < LH) fetch(&tm_k, s_base + oUK + (uint32_t)(s ^ 1) * kTileU, bar_k[s ^ 1], nxt);
      if (need_v) fetch(&tm_v, v_s, bar_v, cur);
    }
    const int64_t lh = cur.lh;
    const int ch = cur.ch;
    const int64_t beg = a.lo + (int64_t)ch * kUC;
    const int64_t eslot = lh * a.edge_stride + (int64_t)ch * kUM;
    int my_deg = 1, ext_b = -1, ext_sel = 0;
    if (a.deg_src && tid < kUC) my_deg = a.deg_src[lh * a.src_cap + beg + tid];
    if (mode == kModeExternal && tid < kUM) {
      ext_b = a.edge_b[eslot + tid];
      ext_sel = a.sel[eslot + tid];
    }
    const int64_t out_base = (mode == kModeExternal) ? (int64_t)a.chunk_out_off[lh * a.n_chunks + ch]
                                                     : a.out_lo + (int64_t)ch * a.out_stride;

    {
      const uint32_t par = (uint32_t)((n >> 1) & 1);
      const bool ok = mbar_wait(bar_k[s], par);
      if (__syncthreads_or(!ok)) {
        bail(bar_k[s], par);
        return;
      }
    }
    if (tid < kUC) {
      degs[tid] = my_deg;
      if (tid & 1) dsum[tid >> 1] = my_deg;  // a cluster starts with its B token's own degree
    }

    if (need_sim) {
      // ---- S = A B^T on the tensor cores: K = 128 in eight steps of 16 (32 bytes inside the 128-byte swizzled row)
      if (tid == 0) {
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t off = (uint32_t)(ks >> 2) * kHalf + (uint32_t)(ks & 3) * 32u;
          umma_bf16(tmem, umma_desc_sw128(k_s + off, 16, 1024), umma_desc_sw128(k_s + 2 * kHalf + off, 16, 1024), umma_idesc(false),
                    ks ? 1u : 0u);
        }
        umma_commit(bar_sim);
      }
      // ---- squared norms from diagonals while the MMA runs: warps 0-7 take 16 B tokens each, warps 8-15 (for the
      //      ranking modes) 16 A tokens each
      {
        const int w8 = warp & 7;
        const bool for_a = warp >= 8;
        if (!for_a || need_cos) {
          float n0[4] = {0.f, 0.f, 0.f, 0.f}, n1[4] = {0.f, 0.f, 0.f, 0.f};
          const uint32_t part = k_s + (for_a ? 0u : 2u * kHalf);
          const int r0 = 16 * w8 + (lane & 7);
#pragma unroll
          for (int kq = 0; kq < 4; ++kq) {
            uint32_t p[4], q[4];
            ldsm_x4(part + sw_off(r0, 4 * kq + (lane >> 3)), p);
            ldsm_x4(part + sw_off(r0 + 8, 4 * kq + (lane >> 3)), q);
            // rows 0-7 <- the first eight tokens, rows 8-15 <- the next eight; columns: the first eight, then the next
            mma_bf16(n0, p[0], q[0], p[1], q[1], p[0], p[1]);
            mma_bf16(n0, p[2], q[2], p[3], q[3], p[2], p[3]);
            mma_bf16(n1, p[0], q[0], p[1], q[1], q[0], q[1]);
            mma_bf16(n1, p[2], q[2], p[3], q[3], q[2], q[3]);
          }
          // the diagonal entry of row r sits in lane 4 r' + r'/2 (r' = r mod 8), register r' & 1 (+2 for rows 8-15)
          if (t == (g >> 1)) {
            const float s0 = (g & 1) ? n0[1] : n0[0], s1 = (g & 1) ? n1[3] : n1[2];
            const int base = (for_a ? 0 : kUM) + 16 * w8;
            inv_nrm[base + g] = s0 > 0.f ? rsqrtf(s0) : 0.f;  // a zero key has similarity 0 with everything
            inv_nrm[base + 8 + g] = s1 > 0.f ? rsqrtf(s1) : 0.f;
          }
        } else if (lane < 16) {
          inv_nrm[16 * w8 + lane] = 1.f;  // the argmax alone does not need |a|
        }
      }
      {
        const bool ok = mbar_wait(bar_sim, ph_sim);
        if (__syncthreads_or(!ok)) {  // also: the norms are visible
          bail(bar_sim, ph_sim);
          return;
        }
        ph_sim ^= 1;
      }
      // ---- Eq. 2 and the row argmax: this thread owns A token 32 (warp % 4) + lane and 32 of the 128 columns
      {
        tc_fence_after();
        const int ai = 32 * (warp & 3) + lane, cq = warp >> 2, c0 = 32 * cq;
        const float inva = inv_nrm[ai];
        float bv = -INFINITY;
        int bi = INT_MAX;
        float v[32];
        tmem_ld32(tmem + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)c0, v);
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const float4 ib = *reinterpret_cast<const float4*>(inv_nrm + kUM + c0 + j);
          const float ibs[4] = {ib.x, ib.y, ib.z, ib.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float sim = v[j + e] * ibs[e] * inva;
            sim += 0.f;  // -0 -> +0, so that the ranking orders zeros as equal
            if (sim > bv) {  // columns in increasing order: the lowest index wins ties
              bv = sim;
              bi = c0 + j + e;
            }
          }
        }
        part_s[ai * 4 + cq] = bv;
        part_b[ai * 4 + cq] = bi;
        tc_fence_before();
      }
    }
    __syncthreads();  // the partial argmaxes are visible; tensor memory columns [0, 128) are free again

    // ---- one edge per A token
    if (tid < kUM) {
      float bv = -INFINITY;
      int bi = -1;
      if (need_sim) {
        bi = INT_MAX;
#pragma unroll
        for (int q = 0; q < 4; ++q) {  // column quarters in increasing order: strict > keeps the lowest index
          const float ps = part_s[4 * tid + q];
          const int pb = part_b[4 * tid + q];
          if (pb != INT_MAX && (bi == INT_MAX || ps > bv)) {
            bv = ps;
            bi = pb;
          }
        }
        if (bi == INT_MAX) bi = -1;
        best_s[tid] = bv;
      } else {
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
      cur = nxt;
      continue;
    }

    // ---- Sec. 5.3: which edges are merged; the A token's column of W
    if (mode == kModeChunkTopM) __syncthreads();  // the ranking reads every edge of the chunk
    if (tid < kUM) {
      int sel = 0;
      const int ai = tid, b = best_b[ai];
      if (b >= 0) {
        if (mode == kModeAll) {
          sel = 1;
        } else if (mode == kModeChunkTopM) {
          const float mine = best_s[ai];
          int rank = 0;  // edges of this chunk ranked before mine: higher similarity, or equal and earlier
          for (int o = 0; o < kUM; ++o) {
            const float other = best_s[o];
            rank += (other > mine || (other == mine && o < ai)) ? 1 : 0;
          }
          sel = rank < a.m_full ? 1 : 0;
        } else {
          sel = ext_sel ? 1 : 0;
        }
      }
      const int da = degs[2 * ai];
      const uint32_t tgt = sel ? (uint32_t)b << 16 : 0xffff0000u;
      tw[ai] = tgt | (__float_as_uint((float)(da & 255)) >> 16);
      tw[kUM + ai] = tgt | (__float_as_uint((float)(da & 0xff00)) >> 16);
      tw[2 * kUM + ai] = tgt | (__float_as_uint((float)(da & 0xff0000)) >> 16);
      if (sel) atomicAdd(&dsum[b], da);
      const uint32_t bits = __ballot_sync(0xffffffffu, sel != 0);
      if (lane == 0) selmask[warp] = bits;
    }
    // do the weights need more than one bf16 piece?  (also: tables visible)
    // (the barrier's reduction is a predicate, not a bitwise OR: ask for the third piece only when a second is needed)
    int n_pieces = 1;
    if (__syncthreads_or(my_deg > 255)) n_pieces = __syncthreads_or(my_deg > 65535) ? 3 : 2;

    // ---- output order: survivors keep their order, a merged A token shares its B token's slot
    auto sel_bit = [&](int ai) { return (selmask[ai >> 5] >> (ai & 31)) & 1u; };
    auto sel_below = [&](int x) {
      int cnt = 0;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int lim = x - 32 * w;
        const uint32_t m = selmask[w];
        cnt += lim >= 32 ? __popc(m) : (lim > 0 ? __popc(m & ((1u << lim) - 1u)) : 0);
      }
      return cnt;
    };
    if (tid < kUC) {
      const int ai = tid >> 1;
      const bool gone = !(tid & 1) && sel_bit(ai);
      const int keeper = gone ? 2 * best_b[ai] + 1 : tid;
      const int op = keeper - sel_below((keeper + 1) >> 1);
      if (!gone) {
        row_of[op] = (unsigned short)(((tid & 1) << 7) | ai);
        newdeg[op] = (tid & 1) ? dsum[ai] : degs[tid];
      }
      if (a.assign) a.assign[lh * a.assign_stride + beg + tid] = (int32_t)(out_base + op);
    }
    const int n_out = kUC - sel_below(kUM);

    // ---- Eq. 5: [merged K | merged V] = W X_A on the tensor cores, 64 A tokens at a time (W is a 128 x 64 operand tile)
    {
      const bool ok = mbar_wait(bar_v, ph_v);
      if (__syncthreads_or(!ok)) {
        bail(bar_v, ph_v);
        return;
      }
      ph_v ^= 1;
    }
    bool first = true;
    for (int piece = 0; piece < n_pieces; ++piece) {
      for (int ah = 0; ah < 2; ++ah) {
#pragma unroll
        for (int i = 0; i < kHalf / 16 / kUThreads; ++i)
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(w_s + (uint32_t)(tid + kUThreads * i) * 16u), "r"(0u) : "memory");
        __syncthreads();
        if (tid < 64) {
          const uint32_t x = tw[piece * kUM + ah * 64 + tid];
          const uint32_t b = x >> 16, wbits = x & 0xffffu;
          if (b != 0xffffu && wbits != 0u) {
            const uint32_t off = b * 128u + ((((uint32_t)tid >> 3) ^ (b & 7u)) << 4) + ((uint32_t)tid & 7u) * 2u;
            asm volatile("st.shared.u16 [%0], %1;" ::"r"(w_s + off), "h"((unsigned short)wbits) : "memory");
          }
        }
        fence_async_smem();  // the tensor core reads W through the asynchronous proxy
        __syncthreads();
        if (tid == 0) {
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint64_t wd = umma_desc_sw128(w_s + 32u * ks, 16, 1024);
            const uint32_t xoff = (uint32_t)(ah * 64 + ks * 16) * 128u;  // rows of the A part = the contraction index
            const uint32_t acc = (first && ks == 0) ? 0u : 1u;
            umma_bf16(tmem + 128, wd, umma_desc_sw128(k_s + xoff, kHalf, 1024), umma_idesc(true), acc);
            umma_bf16(tmem + 256, wd, umma_desc_sw128(v_s + xoff, kHalf, 1024), umma_idesc(true), acc);
          }
          umma_commit(bar_mrg);
        }
        first = false;
        const bool ok = mbar_wait(bar_mrg, ph_mrg);  // W may be rewritten, the accumulators may be read
        if (__syncthreads_or(!ok)) {
          bail(bar_mrg, ph_mrg);
          return;
        }
        ph_mrg ^= 1;
      }
    }

    // ---- epilogue: thread = centroid row b of one tile and one half of its columns: own term, division, rounding;
    //      the centroid replaces the B token's row in the tile; an untouched row stays bit for bit
    {
      tc_fence_after();
      const int b = 32 * (warp & 3) + lane, part = (warp >> 2) & 1, ch2 = warp >> 3;  // K or V tile; columns 64 ch2 .. + 63
      const uint32_t tile_b = (part ? v_s : k_s) + 2 * kHalf;
      const int nb = degs[2 * b + 1], ns = dsum[b];
      const bool merged = ns != nb;
      const float wb = (float)nb, inv = 1.0f / (float)ns;
#pragma unroll 1
      for (int c4 = 2 * ch2; c4 < 2 * ch2 + 2; ++c4) {
        float v[32];
        tmem_ld32(tmem + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(128 * (1 + part) + 32 * c4), v);
        if (merged) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t addr = tile_b + sw_off(b, 4 * c4 + j);
            uint4 x;
            ld_shared_v4(addr, x);
            const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
            uint32_t o[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float lo = fmaf(wb, __uint_as_float(xs[e] << 16), v[8 * j + 2 * e]) * inv;
              const float hi = fmaf(wb, __uint_as_float(xs[e] & 0xffff0000u), v[8 * j + 2 * e + 1]) * inv;
              o[e] = pack_bf16x2(lo, hi);
            }
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
          }
        }
      }
      tc_fence_before();
    }
    fence_async_smem();  // the TMA store reads the tiles through the asynchronous proxy
    __syncthreads();

    // ---- the surviving rows leave
    if (mode == kModeAll) {
      if (tid == 0) {  // every A token merged: the 128 B rows are the output, one contiguous tile per tensor and half
        const int row = (int)out_base;
        tma_store_3d(&tm_ko, 0, row, (int)lh, k_s + 2 * kHalf);
        tma_store_3d(&tm_ko, 64, row, (int)lh, k_s + 3 * kHalf);
        tma_store_3d(&tm_vo, 0, row, (int)lh, v_s + 2 * kHalf);
        tma_store_3d(&tm_vo, 64, row, (int)lh, v_s + 3 * kHalf);
        bulk_commit();
      }
    } else {
      unsigned char* kd = reinterpret_cast<unsigned char*>(a.k_dst) + (lh * a.dst_cap + out_base) * (int64_t)(kUD * 2);
      unsigned char* vd = reinterpret_cast<unsigned char*>(a.v_dst) + (lh * a.dst_cap + out_base) * (int64_t)(kUD * 2);
      const int c16 = tid & 15;
#pragma unroll 2
      for (int op = tid >> 4; op < n_out; op += kUThreads / 16) {
        const int ro = row_of[op];
        const uint32_t off = (uint32_t)(ro >> 7) * 2 * kHalf + sw_off(ro & 127, c16);
        uint4 xk, xv;
        ld_shared_v4(k_s + off, xk);
        ld_shared_v4(v_s + off, xv);
        *reinterpret_cast<uint4*>(kd + (size_t)op * 256 + c16 * 16) = xk;
        *reinterpret_cast<uint4*>(vd + (size_t)op * 256 + c16 * 16) = xv;
      }
    }
    if (tid < n_out) {
      const int64_t di = lh * a.dst_cap + out_base + tid;
      const int dg = newdeg[tid];
      a.deg_dst[di] = dg;
      if (a.logdeg_dst) a.logdeg_dst[di] = logf((float)dg);
    }
    __syncthreads();  // the tiles and tables are free (the store's reads are awaited by the fetching thread)
    cur = nxt;
  }
  if (tid == 0) bulk_wait_read();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ---- the matching alone (first pass of a round ranked per head): a pipeline instead of a chain -------------------
// Nothing but the K tile is needed, so three chunks fit: a TMA warp streams K tiles through a ring of three stages, an
// MMA warp issues S = A B^T for up to four chunks ahead (four tensor-memory slots of 128 columns), and two groups of
// eight consumer warps follow, each on every other chunk: inverse norms from the staged tile (the stage goes back to the
// ring once the group and the MMA have read it), then Eq. 2 and the row argmax from tensor memory, (cosine, target) out.
// Loads, contraction and the two groups' epilogues overlap; the chunk-at-a-time kernel above needs 2.7 us per chunk for
// this, its bytes 1.5 us.
constexpr int kMStages = 3;
constexpr int kMSlots = 4;
constexpr int kMConsumers = 16;
constexpr int kMThreads = (kMConsumers + 2) * 32;
constexpr int oMInv = kMStages * kTileU;             // float [kMSlots][256]: A tokens [0,128), B tokens [128,256)
constexpr int oMPartS = oMInv + kMSlots * 1024;      // float [2 groups][128][2]
constexpr int oMPartB = oMPartS + 2048;              // int   [2 groups][128][2]
constexpr int oMBar = oMPartB + 2048;                // full[3], empty[3], tfull[4], tempty[4]
constexpr int oMFlag = oMBar + 128;                  // int: a consumer's wait gave up
constexpr int oMTmem = oMFlag + 16;
constexpr int kMBytes = oMTmem + 16;

__device__ __forceinline__ void mbar_arrive_one(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// C = 256: an item is one chunk.  C = 128: an item is two consecutive chunks (256 tokens, the same tiles and the same
// 128 x 128 contraction); a row then only looks at the 64 columns of its own chunk, the other half of S is ignored (a
// second chunk past the end of the region reads as zeros and is not written).
template <int C>
__global__ void __launch_bounds__(kMThreads, 1)
match_umma_kernel(const __grid_constant__ CUtensorMap tm_k, const RoundArgs a, const int n_full) {
  static_assert(C == 256 || C == 128, "chunk 256, or pairs of chunks of 128");
  const int n_blk = C == 256 ? n_full : (n_full + 1) / 2;  // items per slab
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + kUAlign - 1) & ~(uintptr_t)(kUAlign - 1));
  const uint32_t s_base = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float* inv_all = reinterpret_cast<float*>(smem + oMInv);
  float* part_s = reinterpret_cast<float*>(smem + oMPartS);
  int* part_b = reinterpret_cast<int*>(smem + oMPartB);
  volatile int* s_failed = reinterpret_cast<volatile int*>(smem + oMFlag);
  auto bar_full = [&](int i) { return s_base + oMBar + 8u * i; };
  auto bar_empty = [&](int i) { return s_base + oMBar + 8u * (kMStages + i); };
  auto bar_tfull = [&](int i) { return s_base + oMBar + 8u * (2 * kMStages + i); };
  auto bar_tempty = [&](int i) { return s_base + oMBar + 8u * (2 * kMStages + kMSlots + i); };
  const int64_t n_items = (int64_t)n_blk * a.LH;
  // this CTA's k-th item is item blockIdx.x + k gridDim.x
  const int64_t my_items = n_items > (int64_t)blockIdx.x ? (n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

  if (tid == 0) {
    for (int i = 0; i < kMStages; ++i) {
      mbar_init(bar_full(i), 1);
      mbar_init(bar_empty(i), 1 + kMConsumers / 2);  // the MMA's commit and every warp of the chunk's group (norms read)
    }
    for (int i = 0; i < kMSlots; ++i) {
      mbar_init(bar_tfull(i), 1);
      mbar_init(bar_tempty(i), kMConsumers / 2);
    }
    *s_failed = 0;
    mbar_init_fence();
  }
  if (warp == 0) tmem_alloc(s_base + oMTmem, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + oMTmem);
  bool failed = false;

  if (warp == kMConsumers) {
    // ------------------------------------------------------------------ TMA warp
    if (lane == 0) {
      for (int64_t k = 0; k < my_items && !failed; ++k) {
        const int64_t item = blockIdx.x + k * gridDim.x;
        const int lh = (int)(item / n_blk), ch = (int)(item % n_blk);
        const int st = (int)(k % kMStages);
        if (!mbar_wait(bar_empty(st), (uint32_t)(((k / kMStages) & 1) ^ 1))) {
          failed = true;
          break;
        }
        const uint32_t dst = s_base + (uint32_t)st * kTileU;
        mbar_arrive_expect_tx(bar_full(st), kTileU);
        tma_load_4d(dst, &tm_k, 0, 0, ch * kUM, lh, bar_full(st));
        tma_load_4d(dst + kHalf, &tm_k, 64, 0, ch * kUM, lh, bar_full(st));
        tma_load_4d(dst + 2 * kHalf, &tm_k, 0, 1, ch * kUM, lh, bar_full(st));
        tma_load_4d(dst + 3 * kHalf, &tm_k, 64, 1, ch * kUM, lh, bar_full(st));
      }
    }
  } else if (warp == kMConsumers + 1) {
    // ------------------------------------------------------------------ MMA warp
    if (lane == 0) {
      for (int64_t k = 0; k < my_items && !failed; ++k) {
        const int st = (int)(k % kMStages), sl = (int)(k % kMSlots);
        if (!mbar_wait(bar_full(st), (uint32_t)((k / kMStages) & 1)) || !mbar_wait(bar_tempty(sl), (uint32_t)(((k / kMSlots) & 1) ^ 1))) {
          failed = true;
          break;
        }
        tc_fence_after();
        const uint32_t k_s = s_base + (uint32_t)st * kTileU;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t off = (uint32_t)(ks >> 2) * kHalf + (uint32_t)(ks & 3) * 32u;
          umma_bf16(tmem + (uint32_t)sl * kUM, umma_desc_sw128(k_s + off, 16, 1024), umma_desc_sw128(k_s + 2 * kHalf + off, 16, 1024),
                    umma_idesc(false), ks ? 1u : 0u);
        }
        umma_commit(bar_empty(st));
        umma_commit(bar_tfull(sl));
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers: group 0 takes the even chunks of
    // this CTA, group 1 the odd ones
    const int g = lane >> 2, t = lane & 3;
    const int grp = warp >> 3, wg = warp & 7, gtid = tid & 255;
    const int q = wg & 3, ch2 = wg >> 2;  // tensor-memory lanes 32 q .. + 31 (A tokens); columns 64 ch2 .. + 63 (B tokens)
    float* gpart_s = part_s + grp * 256;
    int* gpart_b = part_b + grp * 256;
    auto group_sync = [&]() {
      if (grp == 0) {
        asm volatile("bar.sync 1, 256;" ::: "memory");
      } else {
        asm volatile("bar.sync 2, 256;" ::: "memory");
      }
    };
    for (int64_t k = grp; k < my_items; k += 2) {
      const int64_t item = blockIdx.x + k * gridDim.x;
      const int lh = (int)(item / n_blk), ch = (int)(item % n_blk);
      const int st = (int)(k % kMStages), sl = (int)(k % kMSlots);
      float* inv_nrm = inv_all + sl * 256;
      // ---- inverse norms from the staged tile: a warp takes two blocks of 16 tokens (blocks 0-7: A tokens, 8-15: B)
      if (!failed && !mbar_wait(bar_full(st), (uint32_t)((k / kMStages) & 1))) failed = true;
      if (!failed) {
        const uint32_t k_s = s_base + (uint32_t)st * kTileU;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int blk = 2 * wg + half, w8 = blk & 7;
          const bool for_a = blk < 8;
          float n0[4] = {0.f, 0.f, 0.f, 0.f}, n1[4] = {0.f, 0.f, 0.f, 0.f};
          const uint32_t part = k_s + (for_a ? 0u : 2u * kHalf);
          const int r0 = 16 * w8 + (lane & 7);
#pragma unroll
          for (int kq = 0; kq < 4; ++kq) {
            uint32_t p[4], qq[4];
            ldsm_x4(part + sw_off(r0, 4 * kq + (lane >> 3)), p);
            ldsm_x4(part + sw_off(r0 + 8, 4 * kq + (lane >> 3)), qq);
            mma_bf16(n0, p[0], qq[0], p[1], qq[1], p[0], p[1]);
            mma_bf16(n0, p[2], qq[2], p[3], qq[3], p[2], p[3]);
            mma_bf16(n1, p[0], qq[0], p[1], qq[1], qq[0], qq[1]);
            mma_bf16(n1, p[2], qq[2], p[3], qq[3], qq[2], qq[3]);
          }
          if (t == (g >> 1)) {  // the diagonal entries (see the kernel above)
            const float s0 = (g & 1) ? n0[1] : n0[0], s1 = (g & 1) ? n1[3] : n1[2];
            const int base = (for_a ? 0 : kUM) + 16 * w8;
            inv_nrm[base + g] = s0 > 0.f ? rsqrtf(s0) : 0.f;
            inv_nrm[base + 8 + g] = s1 > 0.f ? rsqrtf(s1) : 0.f;
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive_one(bar_empty(st));  // this warp is done with the stage
      }
      if (!failed && !mbar_wait(bar_tfull(sl), (uint32_t)((k / kMSlots) & 1))) failed = true;
      if (failed) *s_failed = 1;
      group_sync();  // every warp's norms are visible
      const int ai = 32 * q + lane;
      if (!failed) {
        tc_fence_after();
        const float inva = inv_nrm[ai];
        float bv = -INFINITY;
        int bi = INT_MAX;
        // columns of this thread: 64 (two loads) at chunk 256; at chunk 128 the 32 columns ch2 of the row's own chunk
        constexpr int NH = C == 256 ? 2 : 1;
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          const int c0 = C == 256 ? 64 * ch2 + 32 * h : 64 * (q >> 1) + 32 * ch2;
          float v[32];
          tmem_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(sl * kUM + c0), v);
          if (h == NH - 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_one(bar_tempty(sl));  // this warp has copied its part of the accumulator
          }
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 ib = *reinterpret_cast<const float4*>(inv_nrm + kUM + c0 + j);
            const float ibs[4] = {ib.x, ib.y, ib.z, ib.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float sim = v[j + e] * ibs[e] * inva;
              sim += 0.f;  // -0 -> +0, so that the ranking orders zeros as equal
              if (sim > bv) {  // columns in increasing order: the lowest index wins ties
                bv = sim;
                bi = c0 + j + e;
              }
            }
          }
        }
        gpart_s[ai * 2 + ch2] = bv;
        gpart_b[ai * 2 + ch2] = bi;
      }
      group_sync();  // the partial argmaxes are visible
      if (*s_failed) {
        failed = true;
        break;
      }
      if (gtid < kUM) {
        float bv = gpart_s[2 * gtid];
        int bi = gpart_b[2 * gtid];
        const float ps = gpart_s[2 * gtid + 1];
        const int pb = gpart_b[2 * gtid + 1];
        if (pb != INT_MAX && (bi == INT_MAX || ps > bv)) {  // the upper column half: strict > keeps the lowest index
          bv = ps;
          bi = pb;
        }
        if (C == 256) {
          const int64_t eslot = (int64_t)lh * a.edge_stride + (int64_t)ch * kUM + gtid;
          a.edge_sim[eslot] = bi == INT_MAX ? -INFINITY : bv;
          a.edge_b[eslot] = bi == INT_MAX ? -1 : 2 * bi + 1;
        } else {
          const int hb = gtid >> 6, chunk = 2 * ch + hb;  // the row's chunk; B indices are local to it
          if (chunk < n_full) {
            const int64_t eslot = (int64_t)lh * a.edge_stride + (int64_t)chunk * 64 + (gtid & 63);
            a.edge_sim[eslot] = bi == INT_MAX ? -INFINITY : bv;
            a.edge_b[eslot] = bi == INT_MAX ? -1 : 2 * (bi - 64 * hb) + 1;
          }
        }
      }
    }
  }
  if (failed && lane == 0) atomicExch(a.status, 1);
  tc_fence_before();
  if (__syncthreads_or(failed)) {
    // copies and MMAs issued before the wait that gave up may still be in flight: they end on their own
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 0) tmem_dealloc(tmem, 512);
}

// ---- host side: tensor maps and launch

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// source view: (column 128, parity 2, token pair, slab) over the middle region's full chunks; box = 64 columns of one
// parity for 128 pairs, 128-byte swizzle
bool make_src_map(CUtensorMap* tm, const void* base, int64_t lo, int64_t pairs, int64_t cap, int LH) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {128, 2, (cuuint64_t)pairs, (cuuint64_t)LH};
  const cuuint64_t strides[3] = {256, 512, (cuuint64_t)cap * 256};
  const cuuint32_t box[4] = {64, 1, 128, 1}, es[4] = {1, 1, 1, 1};
  void* addr = const_cast<unsigned char*>(static_cast<const unsigned char*>(base) + lo * 256);
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, addr, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// destination view: (column 128, row, slab); box = 64 columns x 128 rows
bool make_dst_map(CUtensorMap* tm, void* base, int64_t cap, int LH) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {128, (cuuint64_t)cap, (cuuint64_t)LH};
  const cuuint64_t strides[2] = {256, (cuuint64_t)cap * 256};
  const cuuint32_t box[3] = {64, 128, 1}, es[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool round_umma_supported(const RoundArgs& a, int dtype, int D) {
  // chunk 256 in every mode; chunk 128 for the matching pass of a round ranked per head
  const bool shape = a.chunk == kUC || (a.chunk == 128 && a.mode == kModeMatchOnly);
  return dtype == 1 && D == 128 && shape && a.status != nullptr && encode_tiled_fn() != nullptr;
}

// The full chunks of a round at chunk 256.  A shorter last chunk, if any, is left to the tile kernel.
cudaError_t launch_round_umma(const RoundArgs& a, int64_t n_full, cudaStream_t st) {
  if (n_full <= 0) return cudaSuccess;
  CUtensorMap tm_k, tm_v, tm_ko, tm_vo;
  if (!make_src_map(&tm_k, a.k_src, a.lo, n_full * (a.chunk / 2), a.src_cap, a.LH)) return cudaErrorInvalidValue;
  if (a.mode != kModeMatchOnly) {
    if (!make_src_map(&tm_v, a.v_src, a.lo, n_full * kUM, a.src_cap, a.LH)) return cudaErrorInvalidValue;
    if (!make_dst_map(&tm_ko, a.k_dst, a.dst_cap, a.LH) || !make_dst_map(&tm_vo, a.v_dst, a.dst_cap, a.LH)) return cudaErrorInvalidValue;
  } else {
    tm_v = tm_ko = tm_vo = tm_k;  // never used by the matching alone
  }
  if (a.mode == kModeMatchOnly) {
    const size_t msmem = kMBytes + kUAlign;
    auto kern = a.chunk == kUC ? match_umma_kernel<256> : match_umma_kernel<128>;
    cudaError_t em = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)msmem);
    if (em != cudaSuccess) return em;
    const int64_t items = (a.chunk == kUC ? n_full : (n_full + 1) / 2) * a.LH;
    kern<<<(unsigned)std::min<int64_t>(sm_count(), items), kMThreads, msmem, st>>>(tm_k, a, (int)n_full);
    return cudaGetLastError();
  }
  const size_t smem = kUBytes + kUAlign;
  cudaError_t e = cudaFuncSetAttribute(round_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int64_t ctas = std::min<int64_t>(sm_count(), n_full * a.LH);
  round_umma_kernel<<<(unsigned)ctas, kUThreads, smem, st>>>(tm_k, tm_v, tm_ko, tm_vo, a, (int)n_full);
  return cudaGetLastError();
}

}  // namespace ckv
