// Bipartite Soft Matching without chunks (chunk = 0; Sec. 5.2, the "w/o chunk" ablation of Table 8): every A token
// (1st, 3rd, ... of the middle region) is matched against every B token of the same (layer, head), n^2 d / 4
// multiply-adds per head (Table 1) -- a dense contraction, compute-bound, so it runs as a tensor-core GEMM with the
// argmax fused into the epilogue:
//   bsm_norm_kernel     inverse key norms of the A and B tokens
//   bsm_match_kernel    one CTA per 256 A tokens (two row blocks of 128) walks all B tokens in steps of 256: a TMA warp
//                       streams B tiles (de-interleaving tensor map, 128-byte swizzle) through a ring of two steps, an MMA
//                       warp issues tcgen05.mma 128 x 256 x 16 (the widest shape of one CTA: the least shared-memory
//                       operand traffic per flop) for row block 0, then row block 1, each into its own 256 columns of
//                       tensor memory; sixteen consumer warps copy an accumulator to registers (tcgen05.ld), hand it back
//                       to the tensor core at once and keep a running row argmax of dot / |b| (lowest B position on
//                       ties).  The steps are visited from the tile's own neighbourhood outwards, the four warps of a row
//                       share its running maximum, and groups of sixteen columns whose unscaled bound stays below it are
//                       skipped; the edge (cosine, target) is written at the end
//   select_kernel       the M best edges of the head (shared with the chunked path)
//   bsm_prepare_kernel  prefix counts of the selected edges (output slots) and the number of members per B token
//   bsm_prepare_kernel  also lists the members of every B token
//   bsm_merge_kernel    one warp per surviving token: Eq. 5 over its members, taken from the prepared lists
// bf16, head_dim 128.  Waits are bounded; a role whose wait gives up sets the status word and stops; the others follow.
#include <cuda.h>

#include <algorithm>
#include <climits>
#include <cstdint>

#include "../../include/ckv.h"
#include "ckv_common.cuh"
#include "ckv_internal.h"
#include "ckv_ptx.cuh"

namespace ckv {

namespace {

using namespace ptx;

constexpr int kBD = 128;          // head_dim
constexpr int kBT = 128;          // rows of one MMA, rows of one TMA box
constexpr int kBM = 2 * kBT;      // A tokens per CTA: two row blocks, each with its own accumulator
constexpr int kBN = 2 * kBT;      // B tokens per step (columns of one MMA)
constexpr int kBHalf = kBT * 128; // one swizzled box: 128 rows x 64 columns
constexpr int kBSteps = 2;        // steps of B in flight; a step's tiles are free again once the tensor core has read them
constexpr int kBInvSlots = 4;     // 1/|b| slices of a step (1 KiB each)
constexpr int kBConsumers = 16;   // warps: (quarter of the tensor-memory lanes) x (quarter of the step's columns)
constexpr int kBTmemCols = 2 * kBN;
constexpr int kBThreads = (kBConsumers + 2) * 32;
// Shared memory (1024-byte aligned base): A blocks | B ring | 1/|b| ring | barriers | partial argmaxes | tmem address.
// The B ring is split by column half (dims 0..63 | 64..127), each part holding the 128-row boxes of all steps in order, so
// that the 256 rows of a step are contiguous for the tensor core.
constexpr int oBA = 0;
constexpr int oBB = 4 * kBHalf;
constexpr int kBPart = kBSteps * 2 * kBHalf;  // bytes of one column half of the ring
constexpr int oBInv = oBB + 2 * kBPart;
constexpr int oBBar = oBInv + kBInvSlots * kBN * 4;
constexpr int oBPart = oBBar + 256;
constexpr int oBRowMax = oBPart + kBM * 4 * 8;  // float [kBM]: every row's running maximum over all column quarters
constexpr int oBTmem = oBRowMax + kBM * 4;
constexpr int kBBytes = oBTmem + 16;

struct BsmArgs {
  const __nv_bfloat16* k_src;
  int64_t src_cap, lo;
  int32_t nA, nB;         // A and B tokens of the middle region
  int64_t inv_stride;     // floats per head of inv_a / inv_b (multiple of 256)
  float* inv_a;
  float* inv_b;
  float* edge_sim;        // [LH, edge_stride]
  int32_t* edge_b;        // [LH, edge_stride]  local offset 2 b + 1 of the target
  int64_t edge_stride;
  int32_t* status;
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }

__host__ __device__ constexpr uint32_t bsm_idesc() {  // bf16 x bf16 -> fp32, both K-major, M = 128, N = 256
  return (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)kBN >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ __forceinline__ uint4 ld16(const __nv_bfloat16* p) { return *reinterpret_cast<const uint4*>(p); }
__device__ __forceinline__ void unpack8(const uint4 u, float (&f)[8]) {
  f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
  f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
  f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xffff0000u);
  f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xffff0000u);
}

// inverse norms: a warp takes four consecutive tokens, sixteen lanes (16 bytes each) per token, two tokens per load
__global__ void __launch_bounds__(256) bsm_norm_kernel(const BsmArgs a) {
  const int lh = blockIdx.y, lane = threadIdx.x & 31, half = lane >> 4, c8 = (lane & 15) * 8;
  const int64_t mid = (int64_t)a.nA + a.nB;
  const int64_t o0 = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * 4;
  if (o0 >= mid) return;
  const __nv_bfloat16* base = a.k_src + ((int64_t)lh * a.src_cap + a.lo) * kBD + c8;
  const int64_t t0 = o0 + half, t1 = o0 + 2 + half;  // half 0: the two A tokens, half 1: the two B tokens
  const uint4 z = make_uint4(0, 0, 0, 0);
  const uint4 u0 = t0 < mid ? ld16(base + t0 * kBD) : z, u1 = t1 < mid ? ld16(base + t1 * kBD) : z;
  float x[8], y[8];
  unpack8(u0, x);
  unpack8(u1, y);
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    s0 = fmaf(x[e], x[e], s0);
    s1 = fmaf(y[e], y[e], s1);
  }
#pragma unroll
  for (int d = 8; d >= 1; d >>= 1) {
    s0 += __shfl_xor_sync(0xffffffffu, s0, d);
    s1 += __shfl_xor_sync(0xffffffffu, s1, d);
  }
  if ((lane & 15) == 0) {
    float* out = (half ? a.inv_b : a.inv_a) + (int64_t)lh * a.inv_stride;
    if (t0 < mid) out[t0 >> 1] = s0 > 0.f ? rsqrtf(s0) : 0.f;
    if (t1 < mid) out[t1 >> 1] = s1 > 0.f ? rsqrtf(s1) : 0.f;
  }
}

// tcgen05.ld of 32 columns without the wait, and the wait with the registers as operands (so that no use moves above it)
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,"
      "%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]),
                 "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]),
                 "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]),
                 "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
// two fp32 products in one instruction (round to nearest even, as two scalar multiplies)
__device__ __forceinline__ void mul2(float& x, float& y, uint32_t a0, uint32_t a1, uint64_t b) {
  uint64_t a, d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "r"(a0), "r"(a1));
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  uint32_t lo, hi;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(d));
  x = __uint_as_float(lo);
  y = __uint_as_float(hi);
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Bounded wait for the consumer warps: sixteen warps polling one barrier back to back would take issue slots from the
// warps that feed the tensor core, so a poll that fails is followed by a short sleep at once.
__device__ __forceinline__ bool mbar_wait_sleeping(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(i < 8 ? 100 : 400);
  }
  return false;
}

// max for floats in shared memory (order-preserving views of the bit pattern: as int for v >= 0, as unsigned for v < 0)
__device__ __forceinline__ void atomic_max_float(float* addr, float v) {
  if (v >= 0.f)
    atomicMax(reinterpret_cast<int*>(addr), __float_as_int(v));
  else
    atomicMin(reinterpret_cast<unsigned*>(addr), __float_as_uint(v));
}

// Running row argmax over 64 accumulator columns of one tensor-memory lane per thread: dot products scaled by 1 / |b|.
// Four warps share a row (one per quarter of a step's columns); `shared_max` is the row's running maximum over all of
// them, so that a warp whose columns never hold the row's good matches still knows what it has to beat.
// Sixteen columns at a time.  First a bound that needs no scaling: the largest raw dot product of the sixteen times the
// largest 1 / |b| among them (ginv) is at least every scaled value (fp32 multiplication is monotone), so if that stays
// below the row's maximum in every lane of the warp, the group cannot hold the argmax and is skipped -- the common case
// once the first step is in, because an A token's good matches sit in a few groups near it.  Otherwise: scale, one
// maximum per sixteen columns and one warp vote; only when some lane reaches its row's maximum does the warp look for
// the column (the lowest one that holds the group's maximum; the lowest B position wins ties, also against the
// running one).  What a warp keeps is the argmax over its own columns that can still be the row's: the final
// combination over the four quarters takes the highest value, lowest position.
template <bool RAGGED>
__device__ __forceinline__ void argmax_64(const uint32_t (&r)[2][32], const float* invb, const float (&ginv)[4], int col0, int nB,
                                          float& bv, int& bi, float* shared_max) {
  float thr = fmaxf(bv, *shared_max);  // (a stale value is only a weaker threshold)
#pragma unroll
  for (int h = 0; h < 2; ++h) {
#pragma unroll
    for (int g = 0; g < 32; g += 16) {
      if (!RAGGED) {  // (the last step's columns past the end have no defined 1 / |b|: no shortcut there)
        float d[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) d[e] = __uint_as_float(r[h][g + e]);
        const float rm = max3(max3(max3(d[0], d[1], d[2]), max3(d[3], d[4], d[5]), max3(d[6], d[7], d[8])),
                              max3(max3(d[9], d[10], d[11]), max3(d[12], d[13], d[14]), d[15]), 0.f);
        // rm >= 0 by the last operand: a group of negative dot products is bounded by 0
        if (!__any_sync(0xffffffffu, rm * ginv[2 * h + (g >> 4)] >= thr)) continue;
      }
      float sv[16];
#pragma unroll
      for (int e4 = 0; e4 < 16; e4 += 4) {
        const ulonglong2 ib = *reinterpret_cast<const ulonglong2*>(invb + 32 * h + g + e4);
        mul2(sv[e4], sv[e4 + 1], r[h][g + e4], r[h][g + e4 + 1], ib.x);
        mul2(sv[e4 + 2], sv[e4 + 3], r[h][g + e4 + 2], r[h][g + e4 + 3], ib.y);
      }
      const int col = col0 + 32 * h + g;
      if (RAGGED) {
#pragma unroll
        for (int e = 0; e < 16; ++e) sv[e] = col + e < nB ? sv[e] : -INFINITY;
      }
      const float gm = max3(max3(max3(sv[0], sv[1], sv[2]), max3(sv[3], sv[4], sv[5]), max3(sv[6], sv[7], sv[8])),
                            max3(max3(sv[9], sv[10], sv[11]), max3(sv[12], sv[13], sv[14]), sv[15]), -INFINITY);
      if (__any_sync(0xffffffffu, gm >= thr)) {
        int idx = 15;
#pragma unroll
        for (int e = 14; e >= 0; --e) idx = sv[e] == gm ? e : idx;
        if (gm >= thr && (gm > bv || (gm == bv && col + idx < bi))) {  // the steps are not visited in order: ties by position
          bv = gm;
          bi = col + idx;
          thr = gm;
          atomic_max_float(shared_max, gm);
        }
      }
    }
  }
}

__global__ void __launch_bounds__(kBThreads, 1) bsm_match_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                                                                 const BsmArgs a) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t s_base = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int lh = blockIdx.y, atile = blockIdx.x;
  const int n_steps = (a.nB + kBN - 1) / kBN;
  // barriers: full[step slot][row half of the step] | empty[step slot] | tfull[row block] | tempty[row block] | a | inv[slot]
  auto bar_full = [&](int i) { return s_base + oBBar + 8u * i; };
  auto bar_empty = [&](int i) { return s_base + oBBar + 8u * (2 * kBSteps + i); };
  auto bar_tfull = [&](int m) { return s_base + oBBar + 8u * (3 * kBSteps + m); };
  auto bar_tempty = [&](int m) { return s_base + oBBar + 8u * (3 * kBSteps + 2 + m); };
  const uint32_t bar_a = s_base + oBBar + 8u * (3 * kBSteps + 4);
  auto bar_inv = [&](int i) { return s_base + oBBar + 8u * (3 * kBSteps + 5 + i); };

  if (tid == 0) {
    for (int i = 0; i < 2 * kBSteps; ++i) mbar_init(bar_full(i), 1);
    for (int i = 0; i < kBSteps; ++i) mbar_init(bar_empty(i), 1);  // the MMA's commit
    for (int m = 0; m < 2; ++m) {
      mbar_init(bar_tfull(m), 1);
      mbar_init(bar_tempty(m), kBConsumers);
    }
    mbar_init(bar_a, 1);
    for (int i = 0; i < kBInvSlots; ++i) mbar_init(bar_inv(i), 1);
    mbar_init_fence();
  }
  if (warp == 0) tmem_alloc(s_base + oBTmem, kBTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + oBTmem);
  bool failed = false;
  // The B steps are visited starting with the one that holds this tile's own neighbourhood (B tokens of the same
  // positions as its A tokens) and wrapping around: key similarity decays with distance (the paper's Observations 1 and
  // 2), so the running maxima are close to final after the first step and the bound test of the argmax skips nearly
  // everything that follows.  The result does not depend on the order (ties go to the lowest B position explicitly).
  const int t_first = min(atile * (kBM / kBN), n_steps - 1);
  auto step_of = [&](int t) {
    const int x = t_first + t;
    return x >= n_steps ? x - n_steps : x;
  };

  if (warp == kBConsumers) {
    // ------------------------------------------------------------------ TMA warp: the A blocks once, then the B steps
    if (lane == 0) {
      mbar_arrive_expect_tx(bar_a, 4 * kBHalf);
      for (int m = 0; m < 2; ++m) {  // row block m: tokens atile * 256 + 128 m .. + 127 (zero-filled past the end)
        tma_load_4d(s_base + oBA + (uint32_t)m * 2 * kBHalf, &tm_a, 0, 0, atile * kBM + m * kBT, lh, bar_a);
        tma_load_4d(s_base + oBA + (uint32_t)m * 2 * kBHalf + kBHalf, &tm_a, 64, 0, atile * kBM + m * kBT, lh, bar_a);
      }
      for (int t = 0; t < n_steps && !failed; ++t) {
        const int slot = t % kBSteps;
        if (!mbar_wait(bar_empty(slot), (uint32_t)(((t / kBSteps) & 1) ^ 1))) {
          failed = true;
          break;
        }
        for (int hf = 0; hf < 2; ++hf) {  // B tokens t * 256 + 128 hf .. + 127 (zero-filled past the end)
          const uint32_t dst = s_base + oBB + (uint32_t)(2 * slot + hf) * kBHalf;
          mbar_arrive_expect_tx(bar_full(2 * slot + hf), 2 * kBHalf);
          tma_load_4d(dst, &tm_b, 0, 0, step_of(t) * kBN + hf * kBT, lh, bar_full(2 * slot + hf));
          tma_load_4d(dst + kBPart, &tm_b, 64, 0, step_of(t) * kBN + hf * kBT, lh, bar_full(2 * slot + hf));
        }
        // The slice slot of step t was last read for step t - 4; this fetch runs after the MMAs of step t - 2 completed,
        // which were issued after every consumer warp had copied the accumulators of step t - 3 to registers, and a warp
        // does that only after its argmax over step t - 4.
        const int is = t % kBInvSlots;
        mbar_arrive_expect_tx(bar_inv(is), kBN * 4);
        bulk_load(s_base + oBInv + (uint32_t)is * kBN * 4, a.inv_b + (int64_t)lh * a.inv_stride + (int64_t)step_of(t) * kBN, kBN * 4, bar_inv(is));
      }
    }
  } else if (warp == kBConsumers + 1) {
    // ------------------------------------------------------------------ MMA warp: S = A_m B^T into the accumulator of row block m
    if (lane == 0) {
      failed = !mbar_wait(bar_a, 0);
      for (int t = 0; t < n_steps && !failed; ++t) {
        const int slot = t % kBSteps;
        const uint32_t par = (uint32_t)((t / kBSteps) & 1);
        if (!mbar_wait(bar_full(2 * slot), par) || !mbar_wait(bar_full(2 * slot + 1), par)) {
          failed = true;
          break;
        }
        const uint32_t bt = s_base + oBB + (uint32_t)(2 * slot) * kBHalf;
        for (int m = 0; m < 2; ++m) {
          if (!mbar_wait(bar_tempty(m), (uint32_t)((t & 1) ^ 1))) {  // the consumers are done with this block's last step
            failed = true;
            break;
          }
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = (uint32_t)(ks & 3) * 32u;
            umma_bf16(tmem + (uint32_t)m * kBN, umma_desc_sw128(s_base + oBA + (uint32_t)m * 2 * kBHalf + (uint32_t)(ks >> 2) * kBHalf + off, 16, 1024),
                      umma_desc_sw128(bt + (uint32_t)(ks >> 2) * kBPart + off, 16, 1024), bsm_idesc(), ks ? 1u : 0u);
          }
          umma_commit(bar_tfull(m));  // this block's accumulator is complete
        }
        if (!failed) umma_commit(bar_empty(slot));  // the tensor core has read the step's B tiles
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers: running row argmaxes
    // Every warp serves both row blocks: tensor-memory lanes 32 q .. + 31, columns 64 cq .. + 63 of every step.  It copies
    // its part of an accumulator to registers and hands the accumulator back at once, so that the tensor core refills
    // it while the argmax runs on the registers.
    const int q = warp & 3, cq = warp >> 2;
    float bv[2] = {-INFINITY, -INFINITY};
    int bi[2] = {INT_MAX, INT_MAX};
    float* row_max = reinterpret_cast<float*>(smem + oBRowMax);
    if (tid < kBM) row_max[tid] = -INFINITY;
    asm volatile("bar.sync 1, %0;" ::"n"(kBConsumers * 32) : "memory");
    for (int t = 0; t < n_steps && !failed; ++t) {
      const int is = t % kBInvSlots;
      if (!mbar_wait_sleeping(bar_inv(is), (uint32_t)((t / kBInvSlots) & 1))) {
        failed = true;
        break;
      }
      const float* invb = reinterpret_cast<const float*>(smem + oBInv + is * kBN * 4) + 64 * cq;
      const int col0 = step_of(t) * kBN + 64 * cq;
      // the largest 1 / |b| of each of this warp's four groups of sixteen columns (eight lanes x two values per group)
      float ginv[4];
      {
        const float2 iv = *reinterpret_cast<const float2*>(invb + 2 * lane);
        float gx = fmaxf(iv.x, iv.y);
#pragma unroll
        for (int o = 1; o <= 4; o <<= 1) gx = fmaxf(gx, __shfl_xor_sync(0xffffffffu, gx, o));
#pragma unroll
        for (int k = 0; k < 4; ++k) ginv[k] = __shfl_sync(0xffffffffu, gx, 8 * k);
      }
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        if (!mbar_wait_sleeping(bar_tfull(m), (uint32_t)(t & 1))) {
          failed = true;
          break;
        }
        tc_fence_after();
        uint32_t r[2][32];
        const uint32_t tcol = tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(kBN * m + 64 * cq);
        tmem_ld32_issue(tcol, r[0]);
        tmem_ld32_issue(tcol + 32u, r[1]);
        tmem_ld_wait(r[0]);
        tmem_ld_wait(r[1]);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty(m));
        if (col0 + 64 <= a.nB) {  // only the last step can hold columns that are not B tokens
          argmax_64<false>(r, invb, ginv, col0, a.nB, bv[m], bi[m], row_max + kBT * m + 32 * q + lane);
        } else {
          argmax_64<true>(r, invb, ginv, col0, a.nB, bv[m], bi[m], row_max + kBT * m + 32 * q + lane);
        }
      }
    }
    float* part_s = reinterpret_cast<float*>(smem + oBPart);
    int* part_b = reinterpret_cast<int*>(smem + oBPart + kBM * 4 * 4);
#pragma unroll
    for (int m = 0; m < 2; ++m) {
      part_s[4 * (kBT * m + 32 * q + lane) + cq] = bv[m];
      part_b[4 * (kBT * m + 32 * q + lane) + cq] = bi[m];
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kBConsumers * 32) : "memory");
    if (tid < kBM) {
      const int row = tid, ai = atile * kBM + row;
      if (ai < a.nA && !failed) {
        float s0 = part_s[4 * row];
        int b0 = part_b[4 * row];
#pragma unroll
        for (int c = 1; c < 4; ++c) {  // highest similarity; the lowest B position on ties
          const float s1 = part_s[4 * row + c];
          const int b1 = part_b[4 * row + c];
          if (b1 != INT_MAX && (b0 == INT_MAX || s1 > s0 || (s1 == s0 && b1 < b0))) {
            s0 = s1;
            b0 = b1;
          }
        }
        const bool has = b0 != INT_MAX;
        const float cosv = has ? s0 * a.inv_a[(int64_t)lh * a.inv_stride + ai] + 0.f : -INFINITY;
        a.edge_sim[(int64_t)lh * a.edge_stride + ai] = cosv;
        // (no comparison ever held: not-a-number keys.  The edge still names a real B token, so that a ranking that
        // takes every edge never hands the merge an index outside the head.)
        a.edge_b[(int64_t)lh * a.edge_stride + ai] = has ? 2 * b0 + 1 : 1;
      }
    }
  }
  if (failed && lane == 0) atomicExch(a.status, 1);
  tc_fence_before();
  if (__syncthreads_or(failed)) {
    // A wait gave up: copies and MMAs issued before it may still be in flight.  They finish on their own (nothing they
    // depend on is missing), so give them a millisecond before shared and tensor memory go back.
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 0) tmem_dealloc(tmem, kBTmemCols);
}

// ---- after the ranking: output slots and member counts

struct BsmMergeArgs {
  const __nv_bfloat16* k_src;
  const __nv_bfloat16* v_src;
  const int32_t* deg_src;  // may be null: ones
  __nv_bfloat16* k_dst;
  __nv_bfloat16* v_dst;
  int32_t* deg_dst;
  float* logdeg_dst;       // may be null
  int32_t* assign;         // may be null
  int64_t assign_stride;
  int64_t src_cap, dst_cap, lo;
  int32_t nA, nB;
  const int32_t* edge_b;   // [LH, edge_stride]
  const uint8_t* sel;      // [LH, edge_stride]
  int64_t edge_stride;
  int32_t* selpre;         // [LH, edge_stride + 1] selected edges before A token a (exclusive prefix; last = total)
  int32_t* cnt;            // [LH, cnt_stride]     prepare kernel: member counts, then fill cursors; at the end the member
                           //                      of a B token that has exactly one (else -1)
  int32_t* off;            // [LH, cnt_stride + 1] start of each B token's member list (exclusive prefix of the counts)
  int32_t* list;           // [LH, edge_stride]    member A indices, grouped by B token (order inside a group: arbitrary)
  int64_t cnt_stride;
};

constexpr int kPrepThreads = 1024;
constexpr int kPrepRun = 16;  // A tokens per thread and sweep

__global__ void __launch_bounds__(kPrepThreads) bsm_prepare_kernel(const BsmMergeArgs a) {
  __shared__ int warp_tot[kPrepThreads / 32];
  const int lh = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint8_t* sel = a.sel + (int64_t)lh * a.edge_stride;
  const int32_t* eb = a.edge_b + (int64_t)lh * a.edge_stride;
  int32_t* selpre = a.selpre + (int64_t)lh * (a.edge_stride + 1);
  int32_t* cnt = a.cnt + (int64_t)lh * a.cnt_stride;
  for (int b = tid; b < a.nB; b += kPrepThreads) cnt[b] = 0;
  __syncthreads();
  int run_total = 0;
  for (int base = 0; base < a.nA; base += kPrepThreads * kPrepRun) {
    const int first = base + tid * kPrepRun;
    int local = 0;
    uint32_t bits = 0;
    for (int j = 0; j < kPrepRun; ++j) {
      const int ai = first + j;
      if (ai < a.nA && sel[ai]) {
        bits |= 1u << j;
        ++local;
        atomicAdd(&cnt[eb[ai] >> 1], 1);
      }
    }
    // exclusive prefix of `local` over the block
    int inc = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    const int wt = warp_tot[lane];
    int winc = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += y;
    }
    int before = run_total + __shfl_sync(0xffffffffu, winc - wt, warp) + inc - local;
    run_total += __shfl_sync(0xffffffffu, winc, 31);
    __syncthreads();
    for (int j = 0; j < kPrepRun; ++j) {
      const int ai = first + j;
      if (ai < a.nA) selpre[ai] = before;
      before += (bits >> j) & 1u;
    }
  }
  if (tid == 0) selpre[a.nA] = run_total;
  __syncthreads();  // the counts are complete

  // member lists: offsets = exclusive prefix of the counts, then every selected A token takes a place in its target's list
  int32_t* off = a.off + (int64_t)lh * (a.cnt_stride + 1);
  int32_t* list = a.list + (int64_t)lh * a.edge_stride;
  int off_total = 0;
  for (int base = 0; base < a.nB; base += kPrepThreads * kPrepRun) {
    const int first = base + tid * kPrepRun;
    int local = 0;
    for (int j = 0; j < kPrepRun; ++j) local += first + j < a.nB ? cnt[first + j] : 0;
    int inc = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    const int wt = warp_tot[lane];
    int winc = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += y;
    }
    int before = off_total + __shfl_sync(0xffffffffu, winc - wt, warp) + inc - local;
    off_total += __shfl_sync(0xffffffffu, winc, 31);
    __syncthreads();
    for (int j = 0; j < kPrepRun; ++j) {
      if (first + j < a.nB) {
        off[first + j] = before;
        before += cnt[first + j];
      }
    }
  }
  if (tid == 0) off[a.nB] = off_total;
  __syncthreads();
  for (int ai = tid; ai < a.nA; ai += kPrepThreads) {
    if (sel[ai]) {
      const int b = eb[ai] >> 1;
      list[off[b] + atomicSub(&cnt[b], 1) - 1] = ai;
    }
  }
  __syncthreads();
  // the counters are back at zero: reuse them for "the member of a B token that has exactly one" (the common case of
  // the merge, which then needs no look-up in the list)
  for (int b = tid; b < a.nB; b += kPrepThreads) cnt[b] = off[b + 1] - off[b] == 1 ? list[off[b]] : -1;
}

// Eq. 5, one warp per pair (A token 2i, B token 2i + 1) of the middle region; lanes 0-15 carry the K row and lanes
// 16-31 the V row (16 bytes each), so one load or store instruction moves both.  A merged A token writes nothing, a
// survivor is copied to its slot (the raw bits), a B token with members is replaced by the degree-weighted mean of itself
// and its members (taken from the prepared list and added in position order, so the summation order is fixed; a target
// with more than 32 members scans the head's selected edges instead).
__global__ void __launch_bounds__(128, 16) bsm_merge_kernel(const BsmMergeArgs a) {
  const int lh = blockIdx.y, lane = threadIdx.x & 31, half = lane >> 4, c8 = (lane & 15) * 8;
  const int idx = blockIdx.x * 4 + (threadIdx.x >> 5);
  if (idx >= a.nA) return;
  const uint8_t* sel = a.sel + (int64_t)lh * a.edge_stride;
  const int32_t* eb = a.edge_b + (int64_t)lh * a.edge_stride;
  const int32_t* selpre = a.selpre + (int64_t)lh * (a.edge_stride + 1);
  const int64_t src0 = (int64_t)lh * a.src_cap + a.lo, dst0 = (int64_t)lh * a.dst_cap + a.lo;
  const __nv_bfloat16* src = (half ? a.v_src : a.k_src) + c8;
  __nv_bfloat16* dst = (half ? a.v_dst : a.k_dst) + c8;
  auto slot_b = [&](int b) { return (int64_t)(2 * b + 1) - selpre[b + 1]; };  // A tokens 0 .. b come before B token b
  auto finish = [&](int64_t o, int64_t slot, int n_new) {
    if (lane == 0) {
      a.deg_dst[dst0 + slot] = n_new;
      if (a.logdeg_dst) a.logdeg_dst[dst0 + slot] = logf((float)n_new);
      if (a.assign) a.assign[(int64_t)lh * a.assign_stride + a.lo + o] = (int32_t)(a.lo + slot);
    }
  };
  const int64_t oa = 2 * (int64_t)idx, ob = oa + 1;
  const bool has_b = idx < a.nB;
  const int32_t* off = a.off + (int64_t)lh * (a.cnt_stride + 1);
  // everything that depends on nothing is requested first: flags, slots, list bounds, degree, the B row
  const bool a_merged = sel[idx] != 0;
  const int sp0 = selpre[idx], sp1 = selpre[idx + 1];
  const int l0 = has_b ? off[idx] : 0, l1 = has_b ? off[idx + 1] : 0;
  const int single = has_b ? a.cnt[(int64_t)lh * a.cnt_stride + idx] : -1;
  int n_new = has_b && a.deg_src ? a.deg_src[src0 + ob] : 1;
  const uint4 z = make_uint4(0, 0, 0, 0);
  const uint4 rb = has_b ? ld16(src + (src0 + ob) * kBD) : z;
  const uint4 ra = a_merged ? z : ld16(src + (src0 + oa) * kBD);
  if (a_merged) {
    if (a.assign && lane == 0) a.assign[(int64_t)lh * a.assign_stride + a.lo + oa] = (int32_t)(a.lo + slot_b(eb[idx] >> 1));
  } else {
    const int64_t slot = oa - sp0;
    *reinterpret_cast<uint4*>(dst + (dst0 + slot) * kBD) = ra;
    finish(oa, slot, a.deg_src ? a.deg_src[src0 + oa] : 1);
  }
  if (!has_b) return;
  const int64_t slot = ob - sp1;  // A tokens 0 .. idx come before this B token
  const int m = l1 - l0;
  uint4 out = rb;  // an untouched row keeps its bits
  if (m > 0) {
    float f[8];
    unpack8(rb, f);
    const float wb = (float)n_new;
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] *= wb;
    auto add_member = [&](int am) {
      const int64_t r = src0 + 2 * (int64_t)am;
      float g[8];
      unpack8(ld16(src + r * kBD), g);
      const int wa = a.deg_src ? a.deg_src[r] : 1;
      const float w = (float)wa;
      n_new += wa;
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = fmaf(w, g[e], f[e]);
    };
    if (m == 1) {
      add_member(single);
    } else if (m <= 32) {
      // the list is in arbitrary order: add the members in increasing position, so that the sum is reproducible
      const int mine = lane < m ? a.list[(int64_t)lh * a.edge_stride + l0 + lane] : INT_MAX;
      int rank = 0;
      for (int i = 0; i < m; ++i) rank += __shfl_sync(0xffffffffu, mine, i) < mine ? 1 : 0;
      for (int r = 0; r < m; ++r) {
        const int src_lane = __ffs(__ballot_sync(0xffffffffu, lane < m && rank == r)) - 1;
        add_member(__shfl_sync(0xffffffffu, mine, src_lane));
      }
    } else {
      // a crowded target: scan the head's selected edges in position order
      const int target = 2 * idx + 1;
      int left = m;
      for (int g0 = 0; g0 < a.nA && left > 0; g0 += 32) {
        const int ai = g0 + lane;
        unsigned members = __ballot_sync(0xffffffffu, ai < a.nA && sel[ai] && eb[ai] == target);
        left -= __popc(members);
        while (members) {
          add_member(g0 + __ffs(members) - 1);
          members &= members - 1;
        }
      }
    }
    const float inv = 1.0f / (float)n_new;
    out.x = pack_bf16x2(f[0] * inv, f[1] * inv);
    out.y = pack_bf16x2(f[2] * inv, f[3] * inv);
    out.z = pack_bf16x2(f[4] * inv, f[5] * inv);
    out.w = pack_bf16x2(f[6] * inv, f[7] * inv);
  }
  *reinterpret_cast<uint4*>(dst + (dst0 + slot) * kBD) = out;
  finish(ob, slot, n_new);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn bsm_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

}  // namespace

bool bsm_supported(int dtype, int D) { return dtype == 1 && D == 128 && bsm_encode_fn() != nullptr; }

// workspace of one no-chunk round, in bytes, for LH slabs whose middle region has `mid` tokens
size_t bsm_workspace_bytes(int64_t LH, int64_t mid) {
  const int64_t nA = (mid + 1) / 2, inv_stride = (nA + 255) / 256 * 256;
  return (size_t)LH * (2 * inv_stride * 4 + (nA + 1) * 4 + inv_stride * 4 + (inv_stride + 1) * 4 + nA * 4) + 1024;
}

// Matching, ranking inputs and merge of one no-chunk round.  edge_sim / edge_b / sel: [LH, nA] arrays of the workspace;
// `scratch`: bsm_workspace_bytes.  launch_select runs between match and merge (called by the driver).
cudaError_t launch_bsm_match(const RoundArgs& r, void* scratch, cudaStream_t st) {
  const int64_t mid = r.hi - r.lo;
  BsmArgs a{};
  a.k_src = static_cast<const __nv_bfloat16*>(r.k_src);
  a.src_cap = r.src_cap;
  a.lo = r.lo;
  a.nA = (int32_t)((mid + 1) / 2);
  a.nB = (int32_t)(mid / 2);
  a.inv_stride = ((int64_t)a.nA + 255) / 256 * 256;
  a.inv_a = static_cast<float*>(scratch);
  a.inv_b = a.inv_a + (int64_t)r.LH * a.inv_stride;
  a.edge_sim = r.edge_sim;
  a.edge_b = r.edge_b;
  a.edge_stride = r.edge_stride;
  a.status = r.status;
  bsm_norm_kernel<<<dim3((unsigned)((mid + 31) / 32), (unsigned)r.LH), 256, 0, st>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  // (column, 1, every second token, slab) views of the middle region, one from its first token (A) and one from its second
  // (B), each exactly as long as its side: rows past the end read as zeros and nothing outside the region is touched
  CUtensorMap tm[2];
  for (int side = 0; side < 2; ++side) {
    const cuuint64_t dims[4] = {128, 1, (cuuint64_t)(side ? a.nB : a.nA), (cuuint64_t)r.LH};
    const cuuint64_t strides[3] = {256, 512, (cuuint64_t)r.src_cap * 256};
    const cuuint32_t box[4] = {64, 1, 128, 1}, es[4] = {1, 1, 1, 1};
    void* addr = const_cast<unsigned char*>(reinterpret_cast<const unsigned char*>(r.k_src) + (r.lo + side) * 256);
    if (bsm_encode_fn()(&tm[side], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, addr, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
  }
  const size_t smem = kBBytes + 1024;
  if ((e = cudaFuncSetAttribute(bsm_match_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  bsm_match_kernel<<<dim3((unsigned)((a.nA + kBM - 1) / kBM), (unsigned)r.LH), kBThreads, smem, st>>>(tm[0], tm[1], a);
  return cudaGetLastError();
}

cudaError_t launch_bsm_merge(const RoundArgs& r, void* scratch, cudaStream_t st) {
  const int64_t mid = r.hi - r.lo;
  BsmMergeArgs a{};
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
  a.lo = r.lo;
  a.nA = (int32_t)((mid + 1) / 2);
  a.nB = (int32_t)(mid / 2);
  a.edge_b = r.edge_b;
  a.sel = r.sel;
  a.edge_stride = r.edge_stride;
  const int64_t inv_stride = ((int64_t)a.nA + 255) / 256 * 256;
  a.selpre = reinterpret_cast<int32_t*>(static_cast<float*>(scratch) + 2 * (int64_t)r.LH * inv_stride);
  a.cnt = a.selpre + (int64_t)r.LH * (a.nA + 1);
  a.cnt_stride = inv_stride;
  a.off = a.cnt + (int64_t)r.LH * inv_stride;
  a.list = a.off + (int64_t)r.LH * (inv_stride + 1);
  bsm_prepare_kernel<<<(unsigned)r.LH, kPrepThreads, 0, st>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  bsm_merge_kernel<<<dim3((unsigned)((a.nA + 3) / 4), (unsigned)r.LH), 128, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace ckv
