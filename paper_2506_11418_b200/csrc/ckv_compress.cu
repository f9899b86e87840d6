// Chunked Soft Matching round (general path): one CTA owns one chunk of one (layer, head).
//
//   Sec. 5.2  chunk the middle region, split each chunk alternately into A (even local offsets)
//             and B (odd), cosine similarity of Eq. 2 between A and B keys, one edge per A token
//             to its most similar B token (lowest B position on ties)
//   Sec. 5.3  merge only the selected edges: all of them, the best m of the chunk, or the flags
//             a per-head ranking wrote (select_kernel below)
//   Eq. 5     degree-weighted centroid of K and V at the B token's place, degrees summed;
//             survivors keep their order
//
// This kernel handles every dtype, chunk size and selection mode; the bf16 / chunk-64 /
// ratio-1 case has a faster kernel of its own.
#include <cfloat>
#include <climits>
#include <algorithm>

#include "ckv_common.cuh"
#include "ckv_internal.h"

namespace ckv {

namespace {

constexpr int kRoundThreads = 256;
constexpr int kRoundWarps = kRoundThreads / 32;

template <int D>
struct RoundSmem {
  static constexpr int LDK = D + 4;  // fp32 row stride: consecutive rows shift by 4 banks, so float4 reads of a
                                     // column by consecutive rows are conflict-free
  static size_t bytes(int c) {
    return (size_t)c * LDK * sizeof(float)   // keys as fp32, A rows first then B rows
           + (size_t)c * sizeof(float)       // norms
           + (size_t)c * sizeof(int)         // degrees
           + (size_t)(c / 2) * (sizeof(float) + 2 * sizeof(int))  // best_s, best_b, selflag
           + (size_t)c * sizeof(int);        // outpos
  }
};

template <typename T, int D>
__global__ void __launch_bounds__(kRoundThreads) round_kernel(const RoundArgs a) {
  static_assert(D == 128, "one lane owns four consecutive elements of a row");
  constexpr int LDK = RoundSmem<D>::LDK;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int c = a.chunk;
  const int hc = c >> 1;
  float* Ks = reinterpret_cast<float*>(smem_raw);
  float* nrm = Ks + (size_t)c * LDK;
  int* degs = reinterpret_cast<int*>(nrm + c);
  float* best_s = reinterpret_cast<float*>(degs + c);
  int* best_b = reinterpret_cast<int*>(best_s + hc);
  int* selflag = best_b + hc;
  int* outpos = selflag + hc;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunk_id = a.chunk_first + blockIdx.x;
  const int lh = blockIdx.y;
  const int64_t beg = a.lo + (int64_t)chunk_id * c;
  const int clen = (int)min((int64_t)c, a.hi - beg);
  const int nA = (clen + 1) >> 1, nB = clen >> 1;
  const T* ksrc = reinterpret_cast<const T*>(a.k_src) + ((int64_t)lh * a.src_cap + beg) * D;
  const T* vsrc = reinterpret_cast<const T*>(a.v_src) + ((int64_t)lh * a.src_cap + beg) * D;
  const int64_t eslot = (int64_t)lh * a.edge_stride + (int64_t)chunk_id * hc;
  // smem row of local token o: A tokens (even o) in rows [0, hc), B tokens (odd o) in rows [hc, c)
  auto srow = [hc](int o) { return ((o & 1) ? hc : 0) + (o >> 1); };

  // ---- stage the key tile as fp32, with row norms and degrees
  for (int o = warp; o < clen; o += kRoundWarps) {
    const float4 x = load4(ksrc + (int64_t)o * D + lane * 4);
    *reinterpret_cast<float4*>(Ks + (size_t)srow(o) * LDK + lane * 4) = x;
    const float ss = warp_sum(fmaf(x.x, x.x, fmaf(x.y, x.y, fmaf(x.z, x.z, x.w * x.w))));
    if (lane == 0) nrm[o] = sqrtf(ss);
  }
  for (int o = tid; o < clen; o += kRoundThreads)
    degs[o] = a.deg_src ? a.deg_src[(int64_t)lh * a.src_cap + beg + o] : 1;
  for (int ai = tid; ai < hc; ai += kRoundThreads) {
    best_s[ai] = -INFINITY;
    best_b[ai] = -1;
  }
  __syncthreads();

  // ---- Eq. 2 on the A x B tile and the row argmax (Sec. 5.2)
  if (a.mode == kModeExternal) {
    for (int ai = tid; ai < nA; ai += kRoundThreads) best_b[ai] = a.edge_b[eslot + ai];
  } else if (nB > 0) {
    const int nj = (nB + 31) >> 5;
    for (int a0 = warp * 4; a0 < nA; a0 += kRoundWarps * 4) {
      float acc[4][4];
      int arow[4], brow[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        arow[i] = min(a0 + i, nA - 1);
        brow[i] = hc + min(lane + 32 * i, nB - 1);
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
      }
      for (int d = 0; d < D; d += 4) {
        float4 av[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) av[i] = *reinterpret_cast<const float4*>(Ks + (size_t)arow[i] * LDK + d);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (j < nj) {
            const float4 bv = *reinterpret_cast<const float4*>(Ks + (size_t)brow[j] * LDK + d);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              acc[i][j] = fmaf(av[i].x, bv.x, acc[i][j]);
              acc[i][j] = fmaf(av[i].y, bv.y, acc[i][j]);
              acc[i][j] = fmaf(av[i].z, bv.z, acc[i][j]);
              acc[i][j] = fmaf(av[i].w, bv.w, acc[i][j]);
            }
          }
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int ai = a0 + i;
        if (ai < nA) {
          float bv = -INFINITY;
          int bi = INT_MAX;
          const float na = nrm[2 * ai];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int bj = lane + 32 * j;
            if (j < nj && bj < nB) {
              const float den = na * nrm[2 * bj + 1];
              float s = den > 0.f ? acc[i][j] / den : 0.f;
              s += 0.f;  // -0 -> +0, so that the ranking key orders zeros as equal
              if (s > bv) {
                bv = s;
                bi = bj;
              }
            }
          }
          warp_argmax(bv, bi);
          if (lane == 0) {
            best_s[ai] = bv;
            best_b[ai] = 2 * bi + 1;
          }
        }
      }
    }
  }
  __syncthreads();

  if (a.mode == kModeMatchOnly) {
    for (int ai = tid; ai < hc; ai += kRoundThreads) {
      a.edge_sim[eslot + ai] = best_s[ai];
      a.edge_b[eslot + ai] = best_b[ai];
    }
    return;
  }

  // ---- Sec. 5.3: which edges are merged
  for (int ai = tid; ai < hc; ai += kRoundThreads) {
    int s = 0;
    if (ai < nA && best_b[ai] >= 0) {
      if (a.mode == kModeAll) {
        s = 1;
      } else if (a.mode == kModeChunkTopM) {
        const int m = (clen == c) ? a.m_full : a.m_tail;
        const float mine = best_s[ai];
        int rank = 0;  // edges of this chunk ranked before mine: higher similarity, or equal and earlier
        for (int o = 0; o < nA; ++o) {
          const float other = best_s[o];
          rank += (other > mine || (other == mine && o < ai)) ? 1 : 0;
        }
        s = rank < m ? 1 : 0;
      } else {
        s = a.sel[eslot + ai] ? 1 : 0;
      }
    }
    selflag[ai] = s;
  }
  __syncthreads();

  // ---- order-preserving compaction inside the chunk
  for (int o = tid; o < clen; o += kRoundThreads) {
    int gone = 0;  // merged A tokens before local offset o
    const int na_before = (o + 1) >> 1;
    for (int x = 0; x < na_before; ++x) gone += selflag[x];
    outpos[o] = (!(o & 1) && selflag[o >> 1]) ? -1 : o - gone;
  }
  __syncthreads();

  const int64_t out_base = (a.mode == kModeExternal) ? (int64_t)a.chunk_out_off[(int64_t)lh * a.n_chunks + chunk_id]
                                                     : a.out_lo + (int64_t)chunk_id * a.out_stride;
  T* kdst = reinterpret_cast<T*>(a.k_dst) + ((int64_t)lh * a.dst_cap + out_base) * D;
  T* vdst = reinterpret_cast<T*>(a.v_dst) + ((int64_t)lh * a.dst_cap + out_base) * D;

  // ---- Eq. 5: one warp per surviving token
  for (int o = warp; o < clen; o += kRoundWarps) {
    const int op = outpos[o];
    if (op < 0) continue;
    float4 ak = *reinterpret_cast<const float4*>(Ks + (size_t)srow(o) * LDK + lane * 4);
    float4 av = load4(vsrc + (int64_t)o * D + lane * 4);
    int n_new = degs[o];
    bool merged = false;
    if (o & 1) {
      for (int g = 0; g < nA; g += 32) {
        const int ai = g + lane;
        unsigned mask = __ballot_sync(0xffffffffu, ai < nA && selflag[ai] && best_b[ai] == o);
        while (mask) {
          const int tok = 2 * (g + __ffs(mask) - 1);
          mask &= mask - 1;
          if (!merged) {  // first member: turn the B token's own row into a weighted sum
            merged = true;
            const float wb = (float)n_new;
            ak.x *= wb; ak.y *= wb; ak.z *= wb; ak.w *= wb;
            av.x *= wb; av.y *= wb; av.z *= wb; av.w *= wb;
          }
          const float w = (float)degs[tok];
          const float4 mk = *reinterpret_cast<const float4*>(Ks + (size_t)srow(tok) * LDK + lane * 4);
          const float4 mv = load4(vsrc + (int64_t)tok * D + lane * 4);
          ak.x = fmaf(w, mk.x, ak.x); ak.y = fmaf(w, mk.y, ak.y); ak.z = fmaf(w, mk.z, ak.z); ak.w = fmaf(w, mk.w, ak.w);
          av.x = fmaf(w, mv.x, av.x); av.y = fmaf(w, mv.y, av.y); av.z = fmaf(w, mv.z, av.z); av.w = fmaf(w, mv.w, av.w);
          n_new += degs[tok];
        }
      }
    }
    if (merged) {
      const float n = (float)n_new;
      ak.x /= n; ak.y /= n; ak.z /= n; ak.w /= n;
      av.x /= n; av.y /= n; av.z /= n; av.w /= n;
    }
    store4(kdst + (int64_t)op * D + lane * 4, ak);  // untouched rows round-trip bit-exactly
    store4(vdst + (int64_t)op * D + lane * 4, av);
    if (lane == 0) {
      const int64_t di = (int64_t)lh * a.dst_cap + out_base + op;
      a.deg_dst[di] = n_new;
      if (a.logdeg_dst) a.logdeg_dst[di] = logf((float)n_new);
    }
  }

  if (a.assign) {
    for (int o = tid; o < clen; o += kRoundThreads) {
      const int op = outpos[o] >= 0 ? outpos[o] : outpos[best_b[o >> 1]];
      a.assign[(int64_t)lh * a.assign_stride + beg + o] = (int32_t)(out_base + op);
    }
  }
}

// ---- verbatim copy of token rows (sinks, recent tokens, appended tokens) ---------------------

template <typename T, int D>
__global__ void __launch_bounds__(256) copy_rows_kernel(const CopyArgs a) {
  constexpr int kVecPerRow = D * (int)sizeof(T) / 16;
  if (!a.overlap) griddep_wait();
  griddep_launch();
  const int lh = blockIdx.y;
  const int64_t nvec = a.count * kVecPerRow;
  const uint4* ks = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(a.k_src) + ((int64_t)lh * a.src_cap + a.src_off) * D);
  const uint4* vs = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(a.v_src) + ((int64_t)lh * a.src_cap + a.src_off) * D);
  uint4* kd = reinterpret_cast<uint4*>(reinterpret_cast<T*>(a.k_dst) + ((int64_t)lh * a.dst_cap + a.dst_off) * D);
  uint4* vd = reinterpret_cast<uint4*>(reinterpret_cast<T*>(a.v_dst) + ((int64_t)lh * a.dst_cap + a.dst_off) * D);
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += stride) {
    kd[i] = ks[i];
    vd[i] = vs[i];
  }
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < a.count; i += stride) {
    const int dg = a.deg_src ? a.deg_src[(int64_t)lh * a.src_cap + a.src_off + i] : 1;
    const int64_t di = (int64_t)lh * a.dst_cap + a.dst_off + i;
    a.deg_dst[di] = dg;
    if (a.logdeg_dst) a.logdeg_dst[di] = logf((float)dg);
    if (a.assign) a.assign[(int64_t)lh * a.assign_stride + a.src_off + i] = (int32_t)(a.dst_off + i);
  }
  if (a.overlap) griddep_wait();
}

// Algorithm 1, decoding branch, K = [K, k], V = [V, v], N = [N, 1] for a batch of sequences in one launch: block
// (x, lh) copies the rows of slab lh, one 16-byte piece per thread.
template <typename T, int D>
__global__ void __launch_bounds__(256) append_batch_kernel(const __grid_constant__ AppendBatchArgs a) {
  constexpr int kVecPerRow = D * (int)sizeof(T) / 16;
  griddep_wait();    // ordered launch: the kernel ahead may still be reading the slots this one fills
  griddep_launch();
  const int lh = blockIdx.y;
  const int nvec = a.n * kVecPerRow;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += gridDim.x * blockDim.x) {
    const int b = i / kVecPerRow, piece = i - b * kVecPerRow;
    const int64_t src = ((int64_t)lh * a.n_total + a.first + b) * kVecPerRow + piece;
    const int64_t dst = ((int64_t)lh * a.cap[b] + a.len[b]) * kVecPerRow + piece;
    reinterpret_cast<uint4*>(a.k[b])[dst] = reinterpret_cast<const uint4*>(a.k_new)[src];
    reinterpret_cast<uint4*>(a.v[b])[dst] = reinterpret_cast<const uint4*>(a.v_new)[src];
    if (piece == 0) {
      const int64_t di = (int64_t)lh * a.cap[b] + a.len[b];
      a.deg[b][di] = 1;
      if (a.logdeg[b]) a.logdeg[b][di] = 0.f;
    }
  }
}

// ---- Sec. 5.3, ranking across all chunks of one (layer, head) ---------------------------------
// Exact top-M of the edges by (similarity descending, position ascending): a 4 x 8-bit radix
// select finds the M-th largest similarity, then one pass in position order resolves ties at the
// threshold, writes the selection flags and each chunk's output offset.

__device__ __forceinline__ uint32_t sim_key(float s) {
  const uint32_t b = __float_as_uint(s);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);  // unsigned order == float order
}

constexpr int kSelThreads = 1024;
constexpr int kSelRun = 64;  // edges per thread and sweep of the position-order pass (one bit each in a 64-bit mask)

// exclusive prefix of x over the block, and the block total
__device__ __forceinline__ int block_exscan(int x, int* total, int* warp_tot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  const int wt = warp_tot[lane];  // kSelThreads / 32 == 32 warps: one total per lane
  int winc = wt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, winc, o);
    if (lane >= o) winc += y;
  }
  const int before = __shfl_sync(0xffffffffu, winc - wt, warp);
  *total = __shfl_sync(0xffffffffu, winc, 31);
  __syncthreads();
  return before + inc - x;
}

// STAGED: the head's keys are read from global memory once, into shared memory (one pad word per 32, so that both the
// strided sweeps of the radix passes and the per-thread runs of the position pass are free of bank conflicts); otherwise
// every pass reads them again.
template <bool STAGED>
__global__ void __launch_bounds__(kSelThreads, 2) select_kernel(const SelectArgs a) {
  static_assert(kSelThreads == 1024, "one warp total per lane in block_exscan");
  extern __shared__ uint32_t s_keys[];
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_rem;
  __shared__ int warp_tot[kSelThreads / 32];
  griddep_wait();
  griddep_launch();
  const int tid = threadIdx.x, lane = tid & 31;
  const int lh = blockIdx.x;
  const int64_t n = a.edge_stride;
  const float* sim = a.edge_sim + (int64_t)lh * n;
  const int hc = a.chunk >> 1;
  const bool none = a.M <= 0;
  if (STAGED) {
    const int nn = (int)n;
#pragma unroll 8
    for (int i = tid; i < nn; i += kSelThreads) s_keys[i + (i >> 5)] = sim_key(sim[i]);
    __syncthreads();
  }
  auto key_at = [&](int64_t i) -> uint32_t {
    if (STAGED) return s_keys[(int)i + ((int)i >> 5)];
    return sim_key(sim[i]);
  };

  // ---- the key of the M-th best edge: 4 x 8-bit radix select from the top byte down
  uint32_t prefix = 0, mask = 0, rem = (uint32_t)a.M;
  if (!none) {
    const int64_t n_up = (n + kSelThreads - 1) / kSelThreads * kSelThreads;  // whole warps stay in the loop
    for (int pass = 3; pass >= 0; --pass) {
      const int shift = pass * 8;
      for (int i = tid; i < 256; i += kSelThreads) hist[i] = 0;
      __syncthreads();
      for (int64_t i = tid; i < n_up; i += kSelThreads) {
        const uint32_t key = i < n ? key_at(i) : 0u;
        const bool in = i < n && (key & mask) == prefix;
        const uint32_t bin = in ? ((key >> shift) & 255u) : 256u;
        if (pass == 3) {
          // sign and exponent: similarities cluster, most lanes hit the same bin: one atomic per distinct bin of the warp
          const unsigned peers = __match_any_sync(0xffffffffu, bin);
          if (in && lane == __ffs(peers) - 1) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
        } else if (in) {
          atomicAdd(&hist[bin], 1u);  // mantissa bytes of the few remaining candidates: spread over the bins
        }
      }
      __syncthreads();
      if (tid < 32) {
        // lane L owns bins 255 - 8 L ... 248 - 8 L (descending); find the bin where the count from the top reaches rem
        uint32_t own = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) own += hist[255 - 8 * lane - j];
        uint32_t inc = own;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += y;
        }
        const uint32_t above = inc - own;  // edges in bins above this lane's
        if (above < rem && rem <= inc) {   // exactly one lane
          uint32_t cum = above;
          for (int j = 0; j < 8; ++j) {
            const int bin = 255 - 8 * lane - j;
            const uint32_t h = hist[bin];
            if (cum + h >= rem) {
              s_prefix = prefix | ((uint32_t)bin << shift);
              s_rem = rem - cum;
              break;
            }
            cum += h;
          }
        }
      }
      __syncthreads();
      prefix = s_prefix;
      rem = s_rem;
      mask |= 0xffu << shift;
    }
  }
  const uint32_t T = prefix;   // key of the M-th best edge
  const int quota = (int)rem;  // how many edges equal to T are merged: the earliest ones

  // ---- one pass in position order: every thread owns a run of consecutive edges (all threads busy when the head has
  //      at least 1024 edges; at most 64 per thread and sweep, one bit each in a 64-bit mask)
  const int run = (int)min((int64_t)kSelRun, max((int64_t)1, (n + kSelThreads - 1) / kSelThreads));
  uint8_t* selp = a.sel + (int64_t)lh * n;
  int32_t* offp = a.chunk_out_off + (int64_t)lh * a.n_chunks;
  int sel_run = 0, eq_run = 0;  // totals of the sweeps before this one
  for (int64_t base = 0; base < n; base += (int64_t)kSelThreads * run) {
    const int64_t first = base + (int64_t)tid * run;
    const int len = (int)max((int64_t)0, min((int64_t)run, n - first));
    unsigned long long gt_bits = 0ull, eq_bits = 0ull;
    for (int j = 0; j < len; ++j) {
      const uint32_t key = key_at(first + j);
      if (!none && key > T) gt_bits |= 1ull << j;
      if (!none && key == T) eq_bits |= 1ull << j;
    }
    int eq_tot, s_tot;
    const int eq_ex = eq_run + block_exscan(__popcll(eq_bits), &eq_tot, warp_tot);
    // the earliest `quota` edges equal to the threshold are merged
    const int take = max(0, min(__popcll(eq_bits), quota - eq_ex));
    unsigned long long sel_bits = gt_bits;
    for (unsigned long long e = eq_bits, k = 0; e && (int)k < take; e &= e - 1, ++k) sel_bits |= e & (~e + 1ull);
    const int s_ex = sel_run + block_exscan(__popcll(sel_bits), &s_tot, warp_tot);
    if (len > 0) {
      // flags: four at a time where the run allows it
      if ((len & 3) == 0 && ((reinterpret_cast<uintptr_t>(selp) + (uintptr_t)first) & 3u) == 0) {
        for (int j = 0; j < len; j += 4) {
          const uint32_t nib = (uint32_t)(sel_bits >> j) & 15u;
          *reinterpret_cast<uint32_t*>(selp + first + j) = (nib & 1u) | ((nib & 2u) << 7) | ((nib & 4u) << 14) | ((nib & 8u) << 21);
        }
      } else {
        for (int j = 0; j < len; ++j) selp[first + j] = (uint8_t)((sel_bits >> j) & 1ull);
      }
      // output offset of every chunk that starts inside the run: chunk start minus the edges selected before it
      int64_t ch = (first + hc - 1) / hc;
      for (int64_t at = ch * hc; at < first + len; at += hc, ++ch) {
        const int j = (int)(at - first);
        const int before = s_ex + __popcll(sel_bits & ((1ull << j) - 1ull));
        offp[ch] = (int32_t)(a.lo + ch * a.chunk - before);
      }
    }
    eq_run += eq_tot;
    sel_run += s_tot;
  }
}

__global__ void __launch_bounds__(256) compose_assign_kernel(int32_t* total, const int32_t* step, int64_t n_src,
                                                             int64_t step_stride) {
  griddep_wait();
  griddep_launch();
  const int lh = blockIdx.y;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_src; i += stride) {
    const int64_t at = (int64_t)lh * n_src + i;
    total[at] = step[(int64_t)lh * step_stride + total[at]];
  }
}

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

size_t round_smem_bytes(int chunk, int D) { return D == 128 ? RoundSmem<128>::bytes(chunk) : 0; }

cudaError_t launch_round(const RoundArgs& a, int dtype, int D, cudaStream_t st) {
  if (D != 128) return cudaErrorInvalidValue;
  if (a.n_launch <= 0) return cudaSuccess;
  const size_t smem = RoundSmem<128>::bytes(a.chunk);
  const dim3 grid((unsigned)a.n_launch, (unsigned)a.LH);
  cudaError_t e;
  if (dtype == 0) {
    if ((e = set_smem(round_kernel<float, 128>, smem)) != cudaSuccess) return e;
    round_kernel<float, 128><<<grid, kRoundThreads, smem, st>>>(a);
  } else {
    if ((e = set_smem(round_kernel<__nv_bfloat16, 128>, smem)) != cudaSuccess) return e;
    round_kernel<__nv_bfloat16, 128><<<grid, kRoundThreads, smem, st>>>(a);
  }
  return cudaGetLastError();
}

cudaError_t launch_copy(const CopyArgs& a, int dtype, int D, cudaStream_t st) {
  if (D != 128) return cudaErrorInvalidValue;
  if (a.count <= 0) return cudaSuccess;
  const int64_t nvec = a.count * (D * (dtype == 0 ? 4 : 2) / 16);
  const unsigned gx = (unsigned)std::min<int64_t>((nvec + 255) / 256, 1184);
  const dim3 grid(gx, (unsigned)a.LH);
  return dtype == 0 ? launch_dependent(copy_rows_kernel<float, 128>, grid, dim3(256), 0, st, a)
                    : launch_dependent(copy_rows_kernel<__nv_bfloat16, 128>, grid, dim3(256), 0, st, a);
}

cudaError_t launch_append_batch(const AppendBatchArgs& a, int dtype, int D, cudaStream_t st) {
  if (D != 128) return cudaErrorInvalidValue;
  if (a.n <= 0) return cudaSuccess;
  const int nvec = a.n * (D * (dtype == 0 ? 4 : 2) / 16);
  const dim3 grid((unsigned)((nvec + 255) / 256), (unsigned)a.LH);
  return dtype == 0 ? launch_dependent(append_batch_kernel<float, 128>, grid, dim3(256), 0, st, a)
                    : launch_dependent(append_batch_kernel<__nv_bfloat16, 128>, grid, dim3(256), 0, st, a);
}

cudaError_t launch_select(const SelectArgs& a, cudaStream_t st) {
  // keys of up to 24576 edges per head stay in shared memory (two CTAs of 99 KiB per SM)
  constexpr int64_t kStageMax = 24576;
  if (a.edge_stride <= kStageMax) {
    const size_t smem = (size_t)(a.edge_stride + a.edge_stride / 32 + 1) * 4;
    cudaError_t e = set_smem(select_kernel<true>, (kStageMax + kStageMax / 32 + 1) * 4);
    if (e != cudaSuccess) return e;
    return launch_dependent(select_kernel<true>, dim3((unsigned)a.LH), dim3(kSelThreads), smem, st, a);
  }
  return launch_dependent(select_kernel<false>, dim3((unsigned)a.LH), dim3(kSelThreads), 0, st, a);
}

cudaError_t launch_compose_assign(int32_t* total, const int32_t* step, int64_t n_src, int64_t step_stride, int32_t LH,
                                  cudaStream_t st) {
  if (n_src <= 0) return cudaSuccess;
  const dim3 grid((unsigned)std::min<int64_t>((n_src + 255) / 256, 592), (unsigned)LH);
  return launch_dependent(compose_assign_kernel, grid, dim3(256), 0, st, total, step, n_src, step_stride);
}

}  // namespace ckv
