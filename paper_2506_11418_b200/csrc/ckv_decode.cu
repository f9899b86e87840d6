// Decode attention over the compressed cache (general path), Eq. 3:
//   out = softmax(q K^T * scale + log N) V,   G query heads share one KV head.
// Split-K flash decoding: grid (split, KV head, sequence); each warp walks tiles of 32 tokens of
// its CTA's span with an online softmax, partial (max, sum, out[D]) per split go to the
// workspace and a second kernel combines them.  Scores and sums are fp32 in the exp2 domain.
#include <cfloat>

#include "../../include/ckv.h"
#include "ckv_common.cuh"
#include "ckv_internal.h"

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
  extern __shared__ __align__(16) unsigned char smem_raw[];
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

template <typename T, int D>
__global__ void __launch_bounds__(D / 4) decode_combine_kernel(const DecodeArgs a) {
  const int64_t row = blockIdx.x;  // (b, query head)
  const int lane4 = threadIdx.x;   // four output columns each
  const float* p = a.partial + row * a.n_splits * (D + 4);
  float mm = -INFINITY;
  for (int s = 0; s < a.n_splits; ++s) mm = fmaxf(mm, p[(size_t)s * (D + 4) + D]);
  float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
  float ll = 0.f;
  for (int s = 0; s < a.n_splits; ++s) {
    const float* r = p + (size_t)s * (D + 4);
    const float f = (r[D] == -INFINITY) ? 0.f : exp2f(r[D] - mm);
    const float4 x = *reinterpret_cast<const float4*>(r + lane4 * 4);
    o.x = fmaf(f, x.x, o.x); o.y = fmaf(f, x.y, o.y); o.z = fmaf(f, x.z, o.z); o.w = fmaf(f, x.w, o.w);
    ll = fmaf(f, r[D + 1], ll);
  }
  const float inv = ll > 0.f ? 1.f / ll : 0.f;
  store4(reinterpret_cast<T*>(a.out) + row * D + lane4 * 4, make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv));
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
  decode_combine_kernel<T, D><<<(unsigned)(a.Bz * a.H * G), D / 4, 0, st>>>(a);
  return cudaGetLastError();
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

cudaError_t launch_decode(const DecodeArgs& a, int dtype, int D, cudaStream_t st) {
  if (D != 128) return cudaErrorInvalidValue;
  return dtype == 0 ? launch_decode_t<float>(a, st) : launch_decode_t<__nv_bfloat16>(a, st);
}

}  // namespace ckv

// ---- entry point that allocates nothing ---------------------------------------------------------
// Split partials live in a fixed array inside the library image instead of a caller workspace.
namespace {

constexpr size_t kStaticScratchFloats = (size_t)1 << 20;  // 4 MiB
static __device__ __align__(256) float g_decode_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices];  // device address of g_decode_scratch per device, resolved on first use

}  // namespace

extern "C" int ckv_decode_attn_static(const ckv_layer_view* views_dev, int32_t Bz, int32_t H, int32_t G, int32_t D,
                                      int32_t dtype, const void* q, void* out, float scale, int64_t max_len,
                                      void* cuda_stream) {
  if (!views_dev || !q || !out || Bz <= 0 || H <= 0 || G <= 0 || max_len < 0) return CKV_ERR_INVALID_ARG;
  if (dtype != CKV_F32 && dtype != CKV_BF16) return CKV_ERR_INVALID_ARG;
  if (D != 128 || G > 8 || H > 65535 || Bz > 65535) return CKV_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(q) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u)) return CKV_ERR_ALIGNMENT;
  const int64_t pairs = (int64_t)Bz * H;
  const int64_t max_splits = max_len + 127 > 128 ? (max_len + 127) / 128 : 1;
  int64_t n_splits = (4 * 148 + pairs - 1) / pairs;
  if (n_splits > max_splits) n_splits = max_splits;
  if (n_splits < 1) n_splits = 1;
  // the fixed array bounds the problem size: shrink the split count to fit, reject if even one split does not
  const int64_t per_split = pairs * G * (D + 4);
  if (per_split > (int64_t)kStaticScratchFloats) return CKV_ERR_CAPACITY;
  if (n_splits * per_split > (int64_t)kStaticScratchFloats) n_splits = (int64_t)kStaticScratchFloats / per_split;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CKV_ERR_CUDA;
  if (!g_scratch_ptr[dev]) {
    // In host code `g_decode_scratch` names a host-side shadow of the symbol, not device memory: ask the
    // runtime for the address the array has on the current device and hand that to the kernels.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_decode_scratch) != cudaSuccess || !p) return CKV_ERR_CUDA;
    g_scratch_ptr[dev] = static_cast<float*>(p);
  }
  ckv::DecodeArgs a{};
  a.views = views_dev;
  a.q = q;
  a.out = out;
  a.partial = g_scratch_ptr[dev];
  a.Bz = Bz;
  a.H = H;
  a.G = G;
  a.n_splits = (int32_t)n_splits;
  const int64_t span = ((max_len + n_splits - 1) / n_splits + 127) / 128 * 128;
  a.span = span < 128 ? 128 : span;
  a.scale = scale;
  return ckv::launch_decode(a, dtype, D, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CKV_OK : CKV_ERR_CUDA;
}
