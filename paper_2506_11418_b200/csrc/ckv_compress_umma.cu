// The matching pass of a round ranked per head at chunk 256 (the paper's default) and 128, bf16, head_dim 128, full
// chunks: S = A B^T on the 5th-generation tensor cores (tcgen05.mma) with accumulators in tensor memory, K tiles by TMA.
// Only the K tile is needed, so three chunks fit in shared memory and the pass is a pipeline: a TMA warp streams K tiles
// through a ring of three stages (cp.async.bulk.tensor, 128-byte swizzle; the tensor map views the cache as (column,
// parity, token pair, slab), so the A tokens (1st, 3rd, ...) and the B tokens land de-interleaved, each as two 128 x 64
// operand tiles in the canonical swizzled layout), an MMA warp issues the eight tcgen05.mma of a chunk into one of four
// 128-column tensor-memory slots, and two groups of eight consumer warps follow, each on every other chunk: inverse
// norms from the staged tile (X X^T diagonals with warp-level mma; the stage goes back to the ring once the group and
// the MMA have read it), then tcgen05.ld, the cosine of Eq. 2, the row argmax, (cosine, target) out.
// The rounds that merge run on the warp-group kernel (ckv_compress_group.cu).
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
constexpr int kHalf = kUM * 128;       // one operand tile: 128 rows x 64 columns (128 bytes), swizzled: 16 KiB
constexpr int kTileU = 4 * kHalf;      // A cols 0-63 | A cols 64-127 | B cols 0-63 | B cols 64-127
constexpr int kUAlign = 1024;

// byte offset of element column `col` (0..127) of row `row` inside a part (A or B) of a swizzled tile
__device__ __forceinline__ uint32_t sw_off(int row, int chunk16 /* 0..15: 16-byte piece of the 256-byte row */) {
  return (uint32_t)(chunk16 >> 3) * kHalf + (uint32_t)row * 128u + (uint32_t)(((chunk16 & 7) ^ (row & 7)) << 4);
}

// instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128; b_mn: the B operand is MN-major
__host__ __device__ constexpr uint32_t umma_idesc(bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn ? 1u : 0u) << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

// ---- the pipeline
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
  griddep_wait();    // ordered launch: everything ahead in the stream has completed
  griddep_launch();  // the next launch may become resident as this grid's CTAs leave
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

}  // namespace

bool round_umma_supported(const RoundArgs& a, int dtype, int D) {
  return dtype == 1 && D == 128 && (a.chunk == kUC || a.chunk == 128) && a.mode == kModeMatchOnly && a.status != nullptr &&
         encode_tiled_fn() != nullptr;
}

// The matching pass over the full chunks of a round.  A shorter last chunk, if any, is left to the tile kernel.
cudaError_t launch_round_umma(const RoundArgs& a, int64_t n_full, cudaStream_t st) {
  if (n_full <= 0) return cudaSuccess;
  CUtensorMap tm_k;
  if (!make_src_map(&tm_k, a.k_src, a.lo, n_full * (a.chunk / 2), a.src_cap, a.LH)) return cudaErrorInvalidValue;
  const size_t msmem = kMBytes + kUAlign;
  auto kern = a.chunk == kUC ? match_umma_kernel<256> : match_umma_kernel<128>;
  cudaError_t em = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)msmem);
  if (em != cudaSuccess) return em;
  const int64_t items = (a.chunk == kUC ? n_full : (n_full + 1) / 2) * a.LH;
  return launch_dependent(kern, dim3((unsigned)std::min<int64_t>(sm_count(), items)), dim3(kMThreads), msmem, st, tm_k, a, (int)n_full);
}

}  // namespace ckv
