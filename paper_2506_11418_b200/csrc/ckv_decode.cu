// Decode attention over the compressed cache (general path), Eq. 3:
//   out = softmax(q K^T * scale + log N) V,   G query heads share one KV head.
// Split-K flash decoding: grid (split, KV head, sequence); each warp walks tiles of 32 tokens of
// its CTA's span with an online softmax, partial (max, sum, out[D]) per split go to the
// workspace and a second kernel combines them.  Scores and sums are fp32 in the exp2 domain.
#include <algorithm>
#include <cfloat>

#include "../../include/ckv.h"
#include "ckv_common.cuh"
#include "ckv_internal.h"
#include "ckv_ptx.cuh"

namespace ckv {

namespace {

constexpr int kDecThreads = 128;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kTile = 32;
constexpr int kMaxG = 8;
constexpr float kLog2e = 1.4426950408889634f;

template <typename T, int D>
struct DecodeSmem {
  static constexpr int kRowBytes = D * (int)sizeof(T) + 16;  // padded: lanes reading their own row in 16-byte pieces
                                                              // spread over all banks
  static constexpr size_t kTileBytes = (size_t)kTile * kRowBytes;
  static size_t bytes(int G) {
    return kDecWarps * kTileBytes                       // per-warp K tile
           + (size_t)kDecWarps * kTile * kMaxG * 4      // per-warp probabilities [token][head]
           + (size_t)G * D * 4                          // q as fp32
           + (size_t)kDecWarps * G * (D + 4) * 4;       // per-warp partials for the in-CTA combine
  }
};

// dot of a staged key row (raw dtype, 16-byte pieces) with fp32 q rows in shared memory
template <int D, int G>
__device__ __forceinline__ void row_dot(const float* krow, const float* qs, float* s) {
#pragma unroll 4
  for (int d = 0; d < D; d += 4) {
    const float4 kv = *reinterpret_cast<const float4*>(krow + d);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float4 qv = *reinterpret_cast<const float4*>(qs + g * D + d);
      s[g] = fmaf(kv.x, qv.x, fmaf(kv.y, qv.y, fmaf(kv.z, qv.z, fmaf(kv.w, qv.w, s[g]))));
    }
  }
}

template <int D, int G>
__device__ __forceinline__ void row_dot(const __nv_bfloat16* krow, const float* qs, float* s) {
#pragma unroll 4
  for (int d = 0; d < D; d += 8) {
    const uint4 u = *reinterpret_cast<const uint4*>(krow + d);
    float k[8];
    k[0] = __uint_as_float(u.x << 16); k[1] = __uint_as_float(u.x & 0xffff0000u);
    k[2] = __uint_as_float(u.y << 16); k[3] = __uint_as_float(u.y & 0xffff0000u);
    k[4] = __uint_as_float(u.z << 16); k[5] = __uint_as_float(u.z & 0xffff0000u);
    k[6] = __uint_as_float(u.w << 16); k[7] = __uint_as_float(u.w & 0xffff0000u);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float4 q0 = *reinterpret_cast<const float4*>(qs + g * D + d);
      const float4 q1 = *reinterpret_cast<const float4*>(qs + g * D + d + 4);
      float t = s[g];
      t = fmaf(k[0], q0.x, t); t = fmaf(k[1], q0.y, t); t = fmaf(k[2], q0.z, t); t = fmaf(k[3], q0.w, t);
      t = fmaf(k[4], q1.x, t); t = fmaf(k[5], q1.y, t); t = fmaf(k[6], q1.z, t); t = fmaf(k[7], q1.w, t);
      s[g] = t;
    }
  }
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kDecThreads) decode_split_kernel(const DecodeArgs a) {
  static_assert(D == 128 && G <= kMaxG, "one lane owns four output columns");
  using S = DecodeSmem<T, D>;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  unsigned char* ktile = smem_raw + warp * S::kTileBytes;
  float* probs = reinterpret_cast<float*>(smem_raw + kDecWarps * S::kTileBytes) + warp * kTile * kMaxG;
  float* qs = reinterpret_cast<float*>(smem_raw + kDecWarps * S::kTileBytes) + kDecWarps * kTile * kMaxG;
  float* red = qs + G * D;  // [warp][G][D + 4]: out[D], max, sum, pad (keeps rows 16-byte aligned)

  const ckv_layer_view view = reinterpret_cast<const ckv_layer_view*>(a.views)[b];
  const int64_t len = view.len;
  const T* kbase = reinterpret_cast<const T*>(view.k) + (int64_t)h * view.cap * D;
  const T* vbase = reinterpret_cast<const T*>(view.v) + (int64_t)h * view.cap * D;
  const float* ldbase = view.logdeg ? view.logdeg + (int64_t)h * view.cap : nullptr;

  const T* qsrc = reinterpret_cast<const T*>(a.q) + ((int64_t)b * a.H + h) * G * D;
  for (int i = tid; i < G * D / 4; i += kDecThreads) {
    const float4 x = load4(qsrc + i * 4);
    const float f = a.scale * kLog2e;
    *reinterpret_cast<float4*>(qs + i * 4) = make_float4(x.x * f, x.y * f, x.z * f, x.w * f);
  }
  __syncthreads();

  const int64_t t_begin = min(len, (int64_t)split * a.span);
  const int64_t t_end = min(len, t_begin + a.span);

  float m[G], l[G], acc[G][4];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m[g] = -INFINITY;
    l[g] = 0.f;
    acc[g][0] = acc[g][1] = acc[g][2] = acc[g][3] = 0.f;
  }

  for (int64_t t0 = t_begin + (int64_t)warp * kTile; t0 < t_end; t0 += kDecWarps * kTile) {
    const int nt = (int)min((int64_t)kTile, t_end - t0);
    // stage the K tile: one coalesced row per step
    for (int r = 0; r < nt; ++r) {
      if constexpr (sizeof(T) == 2) {
        const uint2 x = *reinterpret_cast<const uint2*>(kbase + (t0 + r) * D + lane * 4);
        *reinterpret_cast<uint2*>(ktile + (size_t)r * S::kRowBytes + lane * 8) = x;
      } else {
        const uint4 x = *reinterpret_cast<const uint4*>(kbase + (t0 + r) * D + lane * 4);
        *reinterpret_cast<uint4*>(ktile + (size_t)r * S::kRowBytes + lane * 16) = x;
      }
    }
    __syncwarp();
    // scores: lane = token
    float s[G];
#pragma unroll
    for (int g = 0; g < G; ++g) s[g] = 0.f;
    if (lane < nt) {
      row_dot<D, G>(reinterpret_cast<const T*>(ktile + (size_t)lane * S::kRowBytes), qs, s);
      const float bias = ldbase ? ldbase[t0 + lane] * kLog2e : 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) s[g] += bias;
    } else {
#pragma unroll
      for (int g = 0; g < G; ++g) s[g] = -INFINITY;
    }
    float corr[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float m_new = fmaxf(m[g], warp_max(s[g]));  // finite: the tile has at least one token
      corr[g] = exp2f(m[g] - m_new);
      const float p = exp2f(s[g] - m_new);
      l[g] = l[g] * corr[g] + p;                        // per-lane partial sum, reduced at the end
      m[g] = m_new;
      probs[lane * kMaxG + g] = p;
    }
    __syncwarp();
#pragma unroll
    for (int g = 0; g < G; ++g) {
      acc[g][0] *= corr[g]; acc[g][1] *= corr[g]; acc[g][2] *= corr[g]; acc[g][3] *= corr[g];
    }
    // P V: lane owns output columns 4*lane .. 4*lane+3, V rows straight from global memory
#pragma unroll 4
    for (int r = 0; r < nt; ++r) {
      const float4 v = load4(vbase + (t0 + r) * D + lane * 4);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float p = probs[r * kMaxG + g];
        acc[g][0] = fmaf(p, v.x, acc[g][0]);
        acc[g][1] = fmaf(p, v.y, acc[g][1]);
        acc[g][2] = fmaf(p, v.z, acc[g][2]);
        acc[g][3] = fmaf(p, v.w, acc[g][3]);
      }
    }
    __syncwarp();
  }

  // combine the four warps, write this split's partial
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const float lsum = warp_sum(l[g]);
    float* r = red + ((size_t)warp * G + g) * (D + 4);
    *reinterpret_cast<float4*>(r + lane * 4) = make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]);
    if (lane == 0) {
      r[D] = m[g];
      r[D + 1] = lsum;
    }
  }
  __syncthreads();
  for (int g = warp; g < G; g += kDecWarps) {
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) mm = fmaxf(mm, red[((size_t)w * G + g) * (D + 4) + D]);
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    float ll = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float* r = red + ((size_t)w * G + g) * (D + 4);
      const float f = (r[D] == -INFINITY) ? 0.f : exp2f(r[D] - mm);
      const float4 x = *reinterpret_cast<const float4*>(r + lane * 4);
      o.x = fmaf(f, x.x, o.x); o.y = fmaf(f, x.y, o.y); o.z = fmaf(f, x.z, o.z); o.w = fmaf(f, x.w, o.w);
      ll = fmaf(f, r[D + 1], ll);
    }
    float* dst = a.partial + ((((int64_t)b * a.H + h) * G + g) * a.n_splits + split) * (D + 4);
    *reinterpret_cast<float4*>(dst + lane * 4) = o;
    if (lane == 0) {
      dst[D] = mm;
      dst[D + 1] = ll;
    }
  }
}

// Merges the split partials of one query head: out = sum_s 2^(m_s - m) o_s / sum_s 2^(m_s - m) l_s.
// One CTA per (sequence, query head); the four warps take every fourth split, a lane owns four columns.
constexpr int kCombThreads = 128;

template <typename T, int D>
__global__ void __launch_bounds__(kCombThreads) decode_combine_kernel(const DecodeArgs a) {
  static_assert(D == 128, "a lane owns four of the 128 columns");
  constexpr int P = D + 4, W = kCombThreads / 32;
  __shared__ float s_max[W];
  __shared__ float s_sum[W];
  __shared__ float4 s_out[W][32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t row = blockIdx.x;  // (b, query head)
  const int n = a.n_splits;
  griddep_wait();
  griddep_launch();
  const float* p = a.partial + row * n * P;
  float mm = -INFINITY;
  for (int s = tid; s < n; s += kCombThreads) mm = fmaxf(mm, p[(size_t)s * P + D]);
  mm = warp_max(mm);
  if (lane == 0) s_max[warp] = mm;
  __syncthreads();
  mm = fmaxf(fmaxf(s_max[0], s_max[1]), fmaxf(s_max[2], s_max[3]));

  float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
  float ll = 0.f;
#pragma unroll 4
  for (int s = warp; s < n; s += W) {
    const float* r = p + (size_t)s * P;
    const float ms = r[D];
    const float f = (ms == -INFINITY) ? 0.f : exp2f(ms - mm);
    const float4 x = *reinterpret_cast<const float4*>(r + lane * 4);
    o.x = fmaf(f, x.x, o.x); o.y = fmaf(f, x.y, o.y); o.z = fmaf(f, x.z, o.z); o.w = fmaf(f, x.w, o.w);
    ll = fmaf(f, r[D + 1], ll);
  }
  s_out[warp][lane] = o;
  if (lane == 0) s_sum[warp] = ll;
  __syncthreads();
  if (warp == 0) {
    o = s_out[0][lane];
    ll = s_sum[0];
#pragma unroll
    for (int w = 1; w < W; ++w) {
      const float4 x = s_out[w][lane];
      o.x += x.x; o.y += x.y; o.z += x.z; o.w += x.w;
      ll += s_sum[w];
    }
    const float inv = ll > 0.f ? 1.f / ll : 0.f;
    store4(reinterpret_cast<T*>(a.out) + row * D + lane * 4, make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv));
  }
}

template <typename T, int G>
cudaError_t launch_decode_g(const DecodeArgs& a, cudaStream_t st) {
  constexpr int D = 128;
  const size_t smem = DecodeSmem<T, D>::bytes(G);
  cudaError_t e = cudaFuncSetAttribute(decode_split_kernel<T, D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const dim3 grid((unsigned)a.n_splits, (unsigned)a.H, (unsigned)a.Bz);
  decode_split_kernel<T, D, G><<<grid, kDecThreads, smem, st>>>(a);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  return launch_dependent(decode_combine_kernel<T, D>, dim3((unsigned)(a.Bz * a.H * G)), dim3(kCombThreads), 0, st, a);
}

template <typename T>
cudaError_t launch_decode_t(const DecodeArgs& a, cudaStream_t st) {
  switch (a.G) {
    case 1: return launch_decode_g<T, 1>(a, st);
    case 2: return launch_decode_g<T, 2>(a, st);
    case 3: return launch_decode_g<T, 3>(a, st);
    case 4: return launch_decode_g<T, 4>(a, st);
    case 5: return launch_decode_g<T, 5>(a, st);
    case 6: return launch_decode_g<T, 6>(a, st);
    case 7: return launch_decode_g<T, 7>(a, st);
    case 8: return launch_decode_g<T, 8>(a, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

namespace {

// ---- fast path: bf16, tensor cores, warp-private cp.async pipeline ------------------------------------
// Each warp walks its own span of the sequence in tiles of 32 tokens through a 3-stage ring in shared
// memory (K tile, V tile, log-degrees), filled with 16-byte cp.async copies into an XOR-swizzled layout
// so that ldmatrix is conflict-free.  Per tile:
//   S[head, token]   = Q K^T      mma.sync m16n8k16 (heads padded to 16 rows, K through ldmatrix)
//   online softmax in the exp2 domain with the log-degree bias of Eq. 3
//   O^T[d, head]    += V^T P      mma.sync, V through ldmatrix.trans; P is the score accumulator re-packed
//                                 to bf16, already in the layout the B operand needs
// No CTA-wide barrier is used; a warp whose split is empty leaves at once.
//
// Small batches (CL = 8 or 16): the CTAs of one (sequence, KV head) form a thread-block cluster, every warp of the
// cluster is one split, and the partials never leave the chip: each warp parks its partial in its CTA's shared memory,
// and after a cluster barrier every CTA combines 128 / CL output columns of every query head by reading all CTAs'
// partials through distributed shared memory.  One launch per call, no workspace traffic, no combine kernel.

constexpr int kFT = 32;                         // tokens per tile (large batches)
constexpr int kFStages = 3;
constexpr int kFWarps = 4;
constexpr int kFTileBytes = kFT * 256;          // one bf16 tile of K or V
constexpr int kFStageBytes = 2 * kFTileBytes + kFT * 4;
constexpr size_t kFSmemBytes = (size_t)kFWarps * kFStages * kFStageBytes;
// Small batches (cluster launch).  Measured on batch 1 x 8 KV heads x 16416 tokens: 4 warps x 3 stages x 32-token tiles
// 18.5 us per call, 6 warps x 2 stages 20.0 us, 8 warps x 3 stages x 16-token tiles 20.1 us.
constexpr int kCT = 32;
constexpr int kCWarps = 4;
constexpr int kCStages = 3;
constexpr size_t kCSmemBytes = (size_t)kCWarps * kCStages * (2 * kCT * 256 + kCT * 4);

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

using ptx::ldsm_x4;
using ptx::ldsm_x4_trans;

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// a float of the shared memory of CTA `rank` of this cluster, at the offset `local_addr` has in this CTA's window
__device__ __forceinline__ float ld_cluster_f32(uint32_t local_addr, uint32_t rank) {
  uint32_t ra;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
  return v;
}

// PAGED: the cache lives in fixed-size pages, [n_pages, H, page_tokens, D], and a per-sequence block table maps
// logical block i (tokens i * page_tokens ...) to its page; page_tokens is a multiple of the tile, so a tile never
// straddles pages.  Each lane keeps one entry of the table (32 blocks per refill), handed out by shuffle.
template <bool PAGED, int CL, int TT, int NW, int ST>
__global__ void __launch_bounds__(NW * 32, 1) decode_fast_kernel(const DecodeArgs a) {
  constexpr int D = 128;
  constexpr int kTileBytes = TT * 256;                  // one bf16 tile of K or V
  constexpr int kStageBytes = 2 * kTileBytes + TT * 4;  // K tile, V tile, log-degrees
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int split = blockIdx.x * NW + warp;
  griddep_wait();    // the views, the queries and the partial buffer may belong to the kernel ahead in the stream
  griddep_launch();  // the combine kernel may become resident; it waits for this grid before it reads
  if (CL == 0 && split >= a.n_splits) return;  // (in a cluster every warp is a split, and all reach the barriers)
  const int h = blockIdx.y, b = blockIdx.z, G = a.G;
  ckv_layer_view view{};
  const int32_t* table = nullptr;
  if (PAGED) {
    const ckv_paged_view pv = reinterpret_cast<const ckv_paged_view*>(a.views)[b];
    table = pv.block_table;
    view.len = pv.len + (a.k_new ? 1 : 0);  // fused append: the new token is position pv.len
  } else {
    view = reinterpret_cast<const ckv_layer_view*>(a.views)[b];
  }
  const int64_t len = view.len;
  const int64_t new_pos = (PAGED && a.k_new) ? len - 1 : -1;
  const __nv_bfloat16* knew = PAGED ? reinterpret_cast<const __nv_bfloat16*>(a.k_new) + ((int64_t)b * a.H + h) * 128 : nullptr;
  const __nv_bfloat16* vnew = PAGED ? reinterpret_cast<const __nv_bfloat16*>(a.v_new) + ((int64_t)b * a.H + h) * 128 : nullptr;
  // the sequence's own tiles are dealt evenly to the splits (a ragged batch stays balanced)
  const int64_t seq_tiles = (len + TT - 1) / TT;
  const int64_t t_begin = TT * (seq_tiles * split / a.n_splits);
  const int64_t t_end = min(len, TT * (seq_tiles * (split + 1) / a.n_splits));
  const int ntiles = (int)((t_end - t_begin + TT - 1) / TT);
  const __nv_bfloat16* kbase = PAGED ? reinterpret_cast<const __nv_bfloat16*>(a.k_pages)
                                     : reinterpret_cast<const __nv_bfloat16*>(view.k) + (int64_t)h * view.cap * D;
  const __nv_bfloat16* vbase = PAGED ? reinterpret_cast<const __nv_bfloat16*>(a.v_pages)
                                     : reinterpret_cast<const __nv_bfloat16*>(view.v) + (int64_t)h * view.cap * D;
  const float* ldbase = PAGED ? a.logdeg_pages : (view.logdeg ? view.logdeg + (int64_t)h * view.cap : nullptr);
  // paged: block table entries [blk0, blk0 + 32) of this sequence, one per lane
  const int64_t n_blocks = PAGED ? (len + ((int64_t)1 << a.page_shift) - 1) >> a.page_shift : 0;
  int64_t blk0 = PAGED ? t_begin >> a.page_shift : 0;
  int my_page = (PAGED && ntiles > 0 && blk0 + lane < n_blocks) ? table[blk0 + lane] : 0;
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(smem_raw) + (uint32_t)warp * ST * kStageBytes;
  const float* ring_ld = reinterpret_cast<const float*>(smem_raw + (size_t)warp * ST * kStageBytes);

  // query fragments (A operand, rows = heads; rows >= G are zero)
  uint32_t qa[8][2];
  {
    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(reinterpret_cast<const __nv_bfloat16*>(a.q) +
                                                             (((int64_t)b * a.H + h) * G + g) * D);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][0] = g < G ? qrow[8 * ks + t] : 0u;      // elements 16 ks + 2t, +1
      qa[ks][1] = g < G ? qrow[8 * ks + 4 + t] : 0u;  // elements 16 ks + 8 + 2t, +1
    }
  }
  const float sc = a.scale * kLog2e;

  auto issue = [&](int tile) {
    const int64_t t0 = t_begin + (int64_t)tile * TT;
    const uint32_t st = ring + (uint32_t)(tile % ST) * kStageBytes;
    const int c = lane & 15;
    // row0: where the tile's first token sits in the K / V / log-degree arrays; rows of a tile are contiguous
    int64_t row0 = t0;
    if (PAGED) {
      const int64_t blk = t0 >> a.page_shift;
      if (blk >= blk0 + 32) {  // next 32 entries of the table (tiles are issued in order)
        blk0 = blk;
        my_page = blk0 + lane < n_blocks ? table[blk0 + lane] : 0;
      }
      const int page = __shfl_sync(0xffffffffu, my_page, (int)(blk - blk0));
      row0 = (((int64_t)page * a.H + h) << a.page_shift) + (t0 & (((int64_t)1 << a.page_shift) - 1));
    }
#pragma unroll
    for (int i = 0; i < TT / 2; ++i) {
      const int r = (lane >> 4) + 2 * i;
      const bool ok = t0 + r < t_end;
      const int64_t row = ok ? row0 + r : row0;  // clamped address, zero-filled when out of range
      const uint32_t off = (uint32_t)r * 256u + (uint32_t)((c ^ (r & 7)) << 4);
      const bool fresh = PAGED && t0 + r == new_pos;  // the appended token is read from where the caller put it
      cp_async16(st + off, (fresh ? knew : kbase + row * D) + c * 8, ok ? 16u : 0u);
      cp_async16(st + kTileBytes + off, (fresh ? vnew : vbase + row * D) + c * 8, ok ? 16u : 0u);
    }
    if (ldbase) {  // one log-degree per lane; 4-byte copies have no alignment demands on the slab
      // (the appended token has degree 1: its log-degree is the zero fill)
      const bool ok = lane < TT && t0 + lane < t_end && t0 + lane != new_pos;
      if (TT == 32 || lane < TT) cp_async4(st + 2 * kTileBytes + lane * 4, ldbase + (ok ? row0 + lane : row0), ok ? 4u : 0u);
    }
  };

  if (PAGED && new_pos >= t_begin && new_pos < t_end) {
    // K = [K, k], V = [V, v], N = [N, 1]: the warp whose span holds the new position writes it to its page slot
    const int64_t row = (((int64_t)table[new_pos >> a.page_shift] * a.H + h) << a.page_shift) + (new_pos & (((int64_t)1 << a.page_shift) - 1));
    const uint4 x = reinterpret_cast<const uint4*>(lane < 16 ? knew : vnew)[lane & 15];
    reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(lane < 16 ? a.k_pages_w : a.v_pages_w) + row * D)[lane & 15] = x;
    if (lane == 0) {
      a.deg_pages_w[row] = 1;
      if (a.logdeg_pages_w) a.logdeg_pages_w[row] = 0.f;
    }
  }

  float oacc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;  // for head g (this thread's share of the tokens)

#pragma unroll
  for (int i = 0; i < ST - 1; ++i) {
    if (i < ntiles) issue(i);
    cp_async_commit();
  }
  for (int tile = 0; tile < ntiles; ++tile) {
    cp_async_wait<ST - 2>();
    __syncwarp();
    if (tile + ST - 1 < ntiles) issue(tile + ST - 1);
    cp_async_commit();
    const int stage = tile % ST;
    const uint32_t ks_ = ring + (uint32_t)stage * kStageBytes, vs_ = ks_ + kTileBytes;
    const float* lds = ring_ld + (size_t)stage * (kStageBytes / 4) + 2 * kTileBytes / 4;
    const int nt = (int)min((int64_t)TT, t_end - (t_begin + (int64_t)tile * TT));

    // ---- S = Q K^T for 32 tokens: n tile j covers tokens 8j .. 8j+7
    constexpr int NT = TT / 8;  // n tiles of 8 tokens
    float sacc[NT][4];
#pragma unroll
    for (int j = 0; j < NT; ++j) sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f;
#pragma unroll
    for (int kq = 0; kq < 4; ++kq) {
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const int tok = 8 * j + (lane & 7);
        const int chunk = 4 * kq + (lane >> 3);
        uint32_t r[4];
        ldsm_x4(ks_ + (uint32_t)tok * 256u + (uint32_t)((chunk ^ (tok & 7)) << 4), r);
        ptx::mma_bf16(sacc[j], qa[2 * kq][0], 0u, qa[2 * kq][1], 0u, r[0], r[1]);
        ptx::mma_bf16(sacc[j], qa[2 * kq + 1][0], 0u, qa[2 * kq + 1][1], 0u, r[2], r[3]);
      }
    }
    // ---- bias, mask, online softmax (thread holds head g, tokens 8j + 2t, 8j + 2t + 1)
    float p[NT][2];
    float tmax = -INFINITY;
#pragma unroll
    for (int j = 0; j < NT; ++j) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int tok = 8 * j + 2 * t + e;
        float s = sacc[j][e] * sc + (ldbase ? lds[tok] * kLog2e : 0.f);
        s = tok < nt ? s : -INFINITY;
        p[j][e] = s;
        tmax = fmaxf(tmax, s);
      }
    }
    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
    const float m_new = fmaxf(m_run, tmax);
    const float corr = exp2f(m_run - m_new);
    m_run = m_new;
    float psum = 0.f;
    uint32_t pb[NT];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const float p0 = exp2f(p[j][0] - m_new), p1 = exp2f(p[j][1] - m_new);
      psum += p0 + p1;
      pb[j] = pack_bf16x2(p0, p1);
    }
    l_run = l_run * corr + psum;
    // the output accumulator holds heads 2t and 2t+1: fetch their correction factors from quads 2t and 2t+1
    const float c0 = __shfl_sync(0xffffffffu, corr, 8 * t), c1 = __shfl_sync(0xffffffffu, corr, 8 * t + 4);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      oacc[i][0] *= c0; oacc[i][1] *= c1; oacc[i][2] *= c0; oacc[i][3] *= c1;
    }
    // ---- O^T += V^T P: m tile i covers d = 16 i .. 16 i + 15, k step s covers tokens 16 s .. 16 s + 15
#pragma unroll
    for (int s = 0; s < TT / 16; ++s) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int mi = lane >> 3;
        const int tok = 16 * s + 8 * (mi >> 1) + (lane & 7);
        const int chunk = 2 * i + (mi & 1);
        uint32_t r[4];
        ldsm_x4_trans(vs_ + (uint32_t)tok * 256u + (uint32_t)((chunk ^ (tok & 7)) << 4), r);
        ptx::mma_bf16(oacc[i], r[0], r[1], r[2], r[3], pb[2 * s], pb[2 * s + 1]);
      }
    }
  }
  cp_async_wait<0>();

  // ---- this split's partial: out[D], max, sum per query head
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  if constexpr (CL > 0) {
    // ND output columns per combining CTA (a divisor of 32); with 10 CTAs the first 8 combine 16 columns each
    constexpr int P = D + 4, NP = NW * CL, ND = (D % CL == 0 && 32 % (D / CL) == 0) ? D / CL : 16, NPG = 32 / ND, PER = NP / NPG;
    __syncthreads();  // every warp of the CTA is done with its ring: the partials take its place
    float* part = reinterpret_cast<float*>(smem_raw);  // [warp][8 heads][P]
    float* scl = part + NW * 8 * P;               // [warp][NP] weights 2^(m_p - m)
    if (t == 0) {
      part[(warp * 8 + g) * P + D] = m_run;
      part[(warp * 8 + g) * P + D + 1] = l_run;
    }
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      float* dst = part + (warp * 8 + 2 * t + e) * P;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        dst[16 * i + g] = oacc[i][e];
        dst[16 * i + 8 + g] = oacc[i][2 + e];
      }
    }
    cluster_sync_all();
    const uint32_t part_s = (uint32_t)__cvta_generic_to_shared(smem_raw);
    const int d = lane % ND, pg = lane / ND, d0 = (int)blockIdx.x * ND;  // this CTA's columns d0 .. d0 + ND - 1
    for (int head = warp; head < G && (int)blockIdx.x * ND < D; head += NW) {
      constexpr int NK = (NP + 31) / 32;
      static_assert(NP % NPG == 0, "the partials split evenly over the lane groups");
      float mp[NK], lp[NK], mm = -INFINITY;
#pragma unroll
      for (int k = 0; k < NK; ++k) {
        const int pi = lane + 32 * k;  // partial of warp (pi % NW) of CTA (pi / NW)
        const uint32_t addr = part_s + (uint32_t)((((pi % NW) * 8 + head) * P + D) * 4);
        mp[k] = pi < NP ? ld_cluster_f32(addr, (uint32_t)(pi / NW)) : -INFINITY;
        lp[k] = pi < NP ? ld_cluster_f32(addr + 4u, (uint32_t)(pi / NW)) : 0.f;
        mm = fmaxf(mm, mp[k]);
      }
      mm = warp_max(mm);
      float ll = 0.f;
#pragma unroll
      for (int k = 0; k < NK; ++k) {
        const float f = mp[k] == -INFINITY ? 0.f : exp2f(mp[k] - mm);
        if (lane + 32 * k < NP) scl[warp * NP + lane + 32 * k] = f;
        ll = fmaf(f, lp[k], ll);
      }
      ll = warp_sum(ll);
      __syncwarp();
      float acc = 0.f;
#pragma unroll 4
      for (int j = 0; j < PER; ++j) {
        const int pi = pg * PER + j;
        acc = fmaf(scl[warp * NP + pi], ld_cluster_f32(part_s + (uint32_t)((((pi % NW) * 8 + head) * P + d0 + d) * 4), (uint32_t)(pi / NW)),
                   acc);
      }
#pragma unroll
      for (int sft = ND; sft < 32; sft <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
      if (pg == 0) {
        const float inv = ll > 0.f ? 1.f / ll : 0.f;
        reinterpret_cast<__nv_bfloat16*>(a.out)[(((int64_t)b * a.H + h) * G + head) * D + d0 + d] = __float2bfloat16_rn(acc * inv);
      }
      __syncwarp();
    }
    cluster_sync_all();  // nobody leaves while its shared memory may still be read
    return;
  }
  float* pbase = a.partial + ((((int64_t)b * a.H + h) * G) * a.n_splits + split) * (D + 4);
  const int64_t hstride = (int64_t)a.n_splits * (D + 4);
  if (t == 0 && g < G) {
    pbase[g * hstride + D] = m_run;
    pbase[g * hstride + D + 1] = l_run;
  }
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int head = 2 * t + e;
    if (head < G) {
      float* dst = pbase + head * hstride;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        dst[16 * i + g] = oacc[i][e];
        dst[16 * i + 8 + g] = oacc[i][2 + e];
      }
    }
  }
}

template <bool PAGED, int CL>
cudaError_t launch_decode_cluster(DecodeArgs a, cudaStream_t st) {
  // (the kernel's attributes were set by max_active_clusters, which every caller asks first)
  auto kern = decode_fast_kernel<PAGED, CL, kCT, kCWarps, kCStages>;
  a.n_splits = kCWarps * CL;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(CL, (unsigned)a.H, (unsigned)a.Bz);
  cfg.blockDim = dim3(kCWarps * 32);
  cfg.dynamicSmemBytes = kCSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = CL;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

// How many clusters of CL CTAs of the decode kernel the device can hold at once (0: this cluster size cannot be
// scheduled here); asked once per device and kernel.
template <bool PAGED, int CL>
int max_active_clusters() {
  constexpr int kMaxDev = 64;
  static int cached[kMaxDev];  // 0 = not asked yet, else the answer + 1
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return 0;
  if (cached[dev] == 0) {
    auto kern = decode_fast_kernel<PAGED, CL, kCT, kCWarps, kCStages>;
    int n = 0;
    bool ok = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCSmemBytes) == cudaSuccess;
    if (ok && CL > 8) ok = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
    if (ok) {
      cudaLaunchConfig_t cfg{};
      cfg.gridDim = dim3(CL, 1, 1);
      cfg.blockDim = dim3(kCWarps * 32);
      cfg.dynamicSmemBytes = kCSmemBytes;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = CL;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) {
        n = 0;
        cudaGetLastError();  // a refusal here only means "not this cluster size"
      }
    }
    cached[dev] = n + 1;
  }
  return cached[dev] - 1;
}

template <bool PAGED>
cudaError_t launch_decode_fast(const DecodeArgs& a, cudaStream_t st) {
  // Few (sequence, head) pairs: one cluster per pair in a single wave.
  // (short caches too: a call costs about 9 us this way against 18 us for the two dependent kernels below)
  const int64_t pairs = (int64_t)a.Bz * a.H, tiles = (a.max_len + kCT - 1) / kCT;
  // The largest cluster of which `pairs` fit at once (on a B200: 7 of 16 CTAs, 11 of 10, 15 of 8); a short cache does
  // not need more than 8 CTAs.
  if (tiles >= 8 * 8 * kCWarps) {
    if (max_active_clusters<PAGED, 16>() >= pairs) return launch_decode_cluster<PAGED, 16>(a, st);
    if (max_active_clusters<PAGED, 10>() >= pairs) return launch_decode_cluster<PAGED, 10>(a, st);
  }
  if (max_active_clusters<PAGED, 8>() >= pairs) return launch_decode_cluster<PAGED, 8>(a, st);
  static bool attr_set[64];  // per device
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(decode_fast_kernel<PAGED, 0, kFT, kFWarps, kFStages>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFSmemBytes);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const dim3 grid((unsigned)((a.n_splits + kFWarps - 1) / kFWarps), (unsigned)a.H, (unsigned)a.Bz);
  if ((e = launch_dependent(decode_fast_kernel<PAGED, 0, kFT, kFWarps, kFStages>, grid, dim3(kFWarps * 32), kFSmemBytes, st, a)) != cudaSuccess) return e;
  return launch_dependent(decode_combine_kernel<__nv_bfloat16, 128>, dim3((unsigned)(a.Bz * a.H * a.G)), dim3(kCombThreads), 0,
                          st, a);
}

}  // namespace

// How a decode call is split over the sequence: the general kernel takes one span per CTA, the bf16
// kernel one span per warp (four per CTA).
void decode_plan(int32_t Bz, int32_t H, int dtype, int64_t max_len, int64_t max_partial_floats, int32_t G, int32_t D,
                 int32_t* n_splits, int64_t* span) {
  const int64_t pairs = (int64_t)Bz * H, sms = sm_count();
  int64_t ns, gran;
  if (dtype == 1) {
    // One CTA per SM (the rings fill its shared memory), four splits per CTA.  Choose the CTAs per (sequence, head)
    // that minimise waves x (tiles per warp + a fixed cost of about two tile times per CTA), with at least four
    // tiles per warp so that the ring has something to overlap.
    gran = 32;
    const int64_t tiles = std::max<int64_t>(1, (max_len + kFT - 1) / kFT);
    const int64_t max_cpp = std::min<int64_t>(64, std::max<int64_t>(1, tiles / (4 * kFWarps)));
    int64_t best = 1, best_cost = INT64_MAX;
    for (int64_t cpp = 1; cpp <= max_cpp; ++cpp) {
      const int64_t waves = (pairs * cpp + sms - 1) / sms;
      const int64_t per_warp = (tiles + cpp * kFWarps - 1) / (cpp * kFWarps);
      const int64_t cost = waves * (per_warp + 2);
      if (cost < best_cost) {
        best_cost = cost;
        best = cpp;
      }
    }
    ns = best * kFWarps;
  } else {
    gran = 128;
    const int64_t cap = std::max<int64_t>(1, (max_len + 127) / 128);
    ns = std::min(cap, (4 * sms + pairs - 1) / pairs);
  }
  ns = std::max<int64_t>(ns, 1);
  const int64_t per_split = pairs * G * (D + 4);
  if (max_partial_floats > 0 && ns * per_split > max_partial_floats) ns = std::max<int64_t>(1, max_partial_floats / per_split);
  *n_splits = (int32_t)ns;
  *span = std::max<int64_t>(gran, ((max_len + ns - 1) / ns + gran - 1) / gran * gran);
}

size_t decode_partial_floats(int32_t Bz, int32_t H, int32_t G, int32_t D, int64_t max_len) {
  size_t need = 0;
  for (int dtype = 0; dtype < 2; ++dtype) {
    int32_t ns;
    int64_t span;
    decode_plan(Bz, H, dtype, max_len, 0, G, D, &ns, &span);
    need = std::max(need, (size_t)Bz * H * G * ns * (D + 4));
  }
  return need;
}

cudaError_t launch_decode(const DecodeArgs& a, int dtype, int D, cudaStream_t st) {
  if (D != 128) return cudaErrorInvalidValue;
  if (dtype == 1) return launch_decode_fast<false>(a, st);
  return launch_decode_t<float>(a, st);
}

cudaError_t launch_decode_paged(const DecodeArgs& a, cudaStream_t st) { return launch_decode_fast<true>(a, st); }

}  // namespace ckv

// ---- entry point that allocates nothing ---------------------------------------------------------
// Split partials live in a fixed array inside the library image instead of a caller workspace.
namespace {

constexpr size_t kStaticScratchFloats = (size_t)1 << 20;  // 4 MiB
static __device__ __align__(256) float g_decode_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
// device address of g_decode_scratch per device, resolved on first use (atomic: two host threads may make their
// first call on a device at the same time; both would store the same address)
std::atomic<float*> g_scratch_ptr[kMaxDevices];

}  // namespace

extern "C" int ckv_decode_attn_static(const ckv_layer_view* views_dev, int32_t Bz, int32_t H, int32_t G, int32_t D,
                                      int32_t dtype, const void* q, void* out, float scale, int64_t max_len,
                                      void* cuda_stream) {
  if (!views_dev || !q || !out || Bz <= 0 || H <= 0 || G <= 0 || max_len < 0) return CKV_ERR_INVALID_ARG;
  if (dtype != CKV_F32 && dtype != CKV_BF16) return CKV_ERR_INVALID_ARG;
  if (D != 128 || G > 8 || H > 65535 || Bz > 65535) return CKV_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(q) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u)) return CKV_ERR_ALIGNMENT;
  // the fixed array bounds the problem size: fewer sequence splits when the usual count does not fit, rejected if
  // even one split does not
  if ((int64_t)Bz * H * G * (D + 4) > (int64_t)kStaticScratchFloats) return CKV_ERR_CAPACITY;
  int32_t n_splits;
  int64_t span;
  ckv::decode_plan(Bz, H, dtype, max_len, (int64_t)kStaticScratchFloats, G, D, &n_splits, &span);

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CKV_ERR_CUDA;
  float* scratch = g_scratch_ptr[dev].load(std::memory_order_relaxed);
  if (!scratch) {
    // In host code `g_decode_scratch` names a host-side shadow of the symbol, not device memory: ask the
    // runtime for the address the array has on the current device and hand that to the kernels.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_decode_scratch) != cudaSuccess || !p) return CKV_ERR_CUDA;
    scratch = static_cast<float*>(p);
    g_scratch_ptr[dev].store(scratch, std::memory_order_relaxed);
  }
  ckv::DecodeArgs a{};
  a.views = views_dev;
  a.q = q;
  a.out = out;
  a.partial = scratch;
  a.Bz = Bz;
  a.H = H;
  a.G = G;
  a.n_splits = n_splits;
  a.span = span;
  a.max_len = max_len;
  a.scale = scale;
  return ckv::launch_decode(a, dtype, D, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CKV_OK : CKV_ERR_CUDA;
}
