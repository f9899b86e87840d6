// Paged cache support: copies between a sequence's pages ([n_pages, H, page_tokens, D], block table) and a contiguous
// slab [H, cap, D], so that the clustering kernels, which work on contiguous slabs, can serve a block-allocated cache.
#include <algorithm>

#include "../../include/ckv.h"
#include "ckv_common.cuh"
#include "ckv_internal.h"

namespace ckv {
namespace {

struct PageCopyArgs {
  const int32_t* table;
  int64_t len, cap;
  unsigned char* k_pages;
  unsigned char* v_pages;
  int32_t* deg_pages;
  float* logdeg_pages;
  unsigned char* k;
  unsigned char* v;
  int32_t* deg;
  float* logdeg;
  int32_t page_shift, H, row_bytes;
};

// grid (x: row groups, y: KV head); 16 bytes per thread and step.  TO_PAGES: slab -> pages, else pages -> slab.
template <bool TO_PAGES>
__global__ void __launch_bounds__(256) page_copy_kernel(const PageCopyArgs a) {
  const int h = blockIdx.y;
  const int vec_per_row = a.row_bytes / 16;
  const int64_t nvec = a.len * vec_per_row;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t mask = ((int64_t)1 << a.page_shift) - 1;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += stride) {
    const int64_t t = i / vec_per_row;
    const int c = (int)(i - t * vec_per_row);
    const int64_t prow = (((int64_t)a.table[t >> a.page_shift] * a.H + h) << a.page_shift) + (t & mask);
    const int64_t srow = (int64_t)h * a.cap + t;
    uint4* kp = reinterpret_cast<uint4*>(a.k_pages + prow * a.row_bytes) + c;
    uint4* vp = reinterpret_cast<uint4*>(a.v_pages + prow * a.row_bytes) + c;
    uint4* ks = reinterpret_cast<uint4*>(a.k + srow * a.row_bytes) + c;
    uint4* vs = reinterpret_cast<uint4*>(a.v + srow * a.row_bytes) + c;
    if (TO_PAGES) {
      *kp = *ks;
      *vp = *vs;
    } else {
      *ks = *kp;
      *vs = *vp;
    }
  }
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < a.len; t += stride) {
    const int64_t prow = (((int64_t)a.table[t >> a.page_shift] * a.H + h) << a.page_shift) + (t & mask);
    const int64_t srow = (int64_t)h * a.cap + t;
    if (TO_PAGES) {
      const int dg = a.deg ? a.deg[srow] : 1;
      if (a.deg_pages) a.deg_pages[prow] = dg;
      if (a.logdeg_pages) a.logdeg_pages[prow] = logf((float)dg);
    } else {
      const int dg = a.deg_pages ? a.deg_pages[prow] : 1;
      if (a.deg) a.deg[srow] = dg;
      if (a.logdeg) a.logdeg[srow] = logf((float)dg);
    }
  }
}

// grid (x, slab lh): K and V rows 16 bytes per thread and step, then degrees and log-degrees one row per thread
__global__ void __launch_bounds__(256) rows_copy_kernel(const RowsCopyArgs a, const __grid_constant__ PagedArgs pools) {
  const int lh = blockIdx.y;
  const int l = lh / pools.H, h = lh - l * pools.H;
  const int64_t mask = ((int64_t)1 << pools.shift) - 1;
  int64_t dst_off = a.dst_off, count = a.count;
  if (a.begin) {
    dst_off = a.begin[(int64_t)lh * a.begin_stride + a.begin_index];
    count = a.dst_end - dst_off;
  }
  const int64_t src_off = a.src_off + (dst_off - a.dst_off);
  auto row_of = [&](const RowsEnd& e, int64_t pos) -> int64_t {
    return e.table ? ((((int64_t)e.table[pos >> pools.shift] * pools.H + h) << pools.shift) + (pos & mask)) : ((int64_t)lh * e.cap + pos);
  };
  const unsigned char* ks = a.src.table ? pools.k[l] : a.src.k;
  const unsigned char* vs = a.src.table ? pools.v[l] : a.src.v;
  unsigned char* kd = a.dst.table ? pools.k[l] : a.dst.k;
  unsigned char* vd = a.dst.table ? pools.v[l] : a.dst.v;
  const int vec_per_row = a.row_bytes / 16;
  const int64_t nvec = count * vec_per_row, stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += stride) {
    const int64_t t = i / vec_per_row;
    const int c = (int)(i - t * vec_per_row);
    const int64_t sr = row_of(a.src, src_off + t), dr = row_of(a.dst, dst_off + t);
    reinterpret_cast<uint4*>(kd + dr * a.row_bytes)[c] = reinterpret_cast<const uint4*>(ks + sr * a.row_bytes)[c];
    reinterpret_cast<uint4*>(vd + dr * a.row_bytes)[c] = reinterpret_cast<const uint4*>(vs + sr * a.row_bytes)[c];
  }
  const int32_t* ds = a.src.table ? pools.deg[l] : a.src.deg;
  int32_t* dd = a.dst.table ? pools.deg[l] : a.dst.deg;
  float* ld = a.dst.table ? pools.logdeg[l] : a.dst.logdeg;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < count; t += stride) {
    const int dg = (a.src_has_deg && ds) ? ds[row_of(a.src, src_off + t)] : 1;
    const int64_t dr = row_of(a.dst, dst_off + t);
    if (dd) dd[dr] = dg;
    if (ld) ld[dr] = logf((float)dg);
  }
}

inline int page_shift_of(int32_t page_tokens) {
  if (page_tokens < 32 || (page_tokens & (page_tokens - 1))) return -1;
  int s = 0;
  while ((1 << s) < page_tokens) ++s;
  return s;
}

int page_copy(bool to_pages, const PageCopyArgs& a, cudaStream_t st) {
  if (a.len == 0) return CKV_OK;
  const int64_t nvec = a.len * (a.row_bytes / 16);
  const dim3 grid((unsigned)std::min<int64_t>((nvec + 255) / 256, 1184), (unsigned)a.H);
  if (to_pages)
    page_copy_kernel<true><<<grid, 256, 0, st>>>(a);
  else
    page_copy_kernel<false><<<grid, 256, 0, st>>>(a);
  return cudaGetLastError() == cudaSuccess ? CKV_OK : CKV_ERR_CUDA;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

cudaError_t launch_rows_copy(const RowsCopyArgs& a, const PagedArgs& pools, cudaStream_t st) {
  if (a.LH <= 0 || (!a.begin && a.count <= 0)) return cudaSuccess;
  const int64_t rows = a.begin ? 64 : a.count;  // with a device-side start the copy is a chunk's worth at most
  const int64_t nvec = rows * (a.row_bytes / 16);
  const dim3 grid((unsigned)std::min<int64_t>((nvec + 255) / 256, 1184), (unsigned)a.LH);
  rows_copy_kernel<<<grid, 256, 0, st>>>(a, pools);
  return cudaGetLastError();
}

int page_shift(int32_t page_tokens) { return page_shift_of(page_tokens); }

}  // namespace ckv

using namespace ckv;

extern "C" {

int ckv_pages_gather(const int32_t* block_table, int64_t len, const void* k_pages, const void* v_pages, const int32_t* deg_pages,
                     int32_t page_tokens, int32_t H, int32_t D, int32_t dtype, void* k, void* v, int32_t* deg, float* logdeg,
                     int64_t cap, void* cuda_stream) {
  if (!block_table || !k_pages || !v_pages || !k || !v || len < 0 || H <= 0 || H > 65535 || cap < len) return CKV_ERR_INVALID_ARG;
  if (dtype != CKV_F32 && dtype != CKV_BF16) return CKV_ERR_INVALID_ARG;
  const int shift = page_shift_of(page_tokens);
  if (shift < 0 || D != 128) return CKV_ERR_UNSUPPORTED;
  if (!aligned16(k_pages) || !aligned16(v_pages) || !aligned16(k) || !aligned16(v)) return CKV_ERR_ALIGNMENT;
  PageCopyArgs a{};
  a.table = block_table; a.len = len; a.cap = cap;
  a.k_pages = static_cast<unsigned char*>(const_cast<void*>(k_pages));
  a.v_pages = static_cast<unsigned char*>(const_cast<void*>(v_pages));
  a.deg_pages = const_cast<int32_t*>(deg_pages);
  a.k = static_cast<unsigned char*>(k); a.v = static_cast<unsigned char*>(v); a.deg = deg; a.logdeg = logdeg;
  a.page_shift = shift; a.H = H; a.row_bytes = D * (dtype == CKV_F32 ? 4 : 2);
  return page_copy(false, a, static_cast<cudaStream_t>(cuda_stream));
}

int ckv_pages_scatter(const int32_t* block_table, int64_t len, const void* k, const void* v, const int32_t* deg, int64_t cap,
                      int32_t page_tokens, int32_t H, int32_t D, int32_t dtype, void* k_pages, void* v_pages, int32_t* deg_pages,
                      float* logdeg_pages, void* cuda_stream) {
  if (!block_table || !k_pages || !v_pages || !k || !v || len < 0 || H <= 0 || H > 65535 || cap < len) return CKV_ERR_INVALID_ARG;
  if (dtype != CKV_F32 && dtype != CKV_BF16) return CKV_ERR_INVALID_ARG;
  const int shift = page_shift_of(page_tokens);
  if (shift < 0 || D != 128) return CKV_ERR_UNSUPPORTED;
  if (!aligned16(k_pages) || !aligned16(v_pages) || !aligned16(k) || !aligned16(v)) return CKV_ERR_ALIGNMENT;
  PageCopyArgs a{};
  a.table = block_table; a.len = len; a.cap = cap;
  a.k_pages = static_cast<unsigned char*>(k_pages); a.v_pages = static_cast<unsigned char*>(v_pages);
  a.deg_pages = deg_pages; a.logdeg_pages = logdeg_pages;
  a.k = static_cast<unsigned char*>(const_cast<void*>(k)); a.v = static_cast<unsigned char*>(const_cast<void*>(v));
  a.deg = const_cast<int32_t*>(deg);
  a.page_shift = shift; a.H = H; a.row_bytes = D * (dtype == CKV_F32 ? 4 : 2);
  return page_copy(true, a, static_cast<cudaStream_t>(cuda_stream));
}

int ckv_decode_attn_paged(const ckv_paged_view* views_dev, const void* k_pages, const void* v_pages, const float* logdeg_pages,
                          int32_t page_tokens, int32_t Bz, int32_t H, int32_t G, int32_t D, int32_t dtype, const void* q,
                          void* out, float scale, int64_t max_len, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!views_dev || !k_pages || !v_pages || !q || !out || Bz <= 0 || H <= 0 || G <= 0 || max_len < 0) return CKV_ERR_INVALID_ARG;
  if (dtype != CKV_F32 && dtype != CKV_BF16) return CKV_ERR_INVALID_ARG;
  const int shift = page_shift_of(page_tokens);
  if (dtype != CKV_BF16 || shift < 0 || D != 128 || G > 8 || H > 65535 || Bz > 65535) return CKV_ERR_UNSUPPORTED;
  if (!aligned16(q) || !aligned16(out) || !aligned16(k_pages) || !aligned16(v_pages)) return CKV_ERR_ALIGNMENT;
  const size_t need = ckv_decode_workspace_bytes(Bz, H, G, D, max_len);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return CKV_ERR_WORKSPACE;
  DecodeArgs a{};
  a.views = views_dev; a.q = q; a.out = out;
  a.partial = static_cast<float*>(workspace);
  a.Bz = Bz; a.H = H; a.G = G;
  decode_plan(Bz, H, dtype, max_len, 0, G, D, &a.n_splits, &a.span);
  a.max_len = max_len;
  a.scale = scale;
  a.k_pages = k_pages; a.v_pages = v_pages; a.logdeg_pages = logdeg_pages; a.page_shift = shift;
  return launch_decode_paged(a, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CKV_OK : CKV_ERR_CUDA;
}

int ckv_decode_append_attn_paged(const ckv_paged_view* views_dev, void* k_pages, void* v_pages, int32_t* deg_pages,
                                 float* logdeg_pages, int32_t page_tokens, int32_t Bz, int32_t H, int32_t G, int32_t D, int32_t dtype,
                                 const void* k_new, const void* v_new, const void* q, void* out, float scale, int64_t max_len,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!views_dev || !k_pages || !v_pages || !deg_pages || !k_new || !v_new || !q || !out || Bz <= 0 || H <= 0 || G <= 0 || max_len < 1)
    return CKV_ERR_INVALID_ARG;
  if (dtype != CKV_F32 && dtype != CKV_BF16) return CKV_ERR_INVALID_ARG;
  const int shift = page_shift_of(page_tokens);
  if (dtype != CKV_BF16 || shift < 0 || D != 128 || G > 8 || H > 65535 || Bz > 65535) return CKV_ERR_UNSUPPORTED;
  if (!aligned16(q) || !aligned16(out) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(k_new) || !aligned16(v_new))
    return CKV_ERR_ALIGNMENT;
  const size_t need = ckv_decode_workspace_bytes(Bz, H, G, D, max_len);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return CKV_ERR_WORKSPACE;
  DecodeArgs a{};
  a.views = views_dev; a.q = q; a.out = out;
  a.partial = static_cast<float*>(workspace);
  a.Bz = Bz; a.H = H; a.G = G;
  decode_plan(Bz, H, dtype, max_len, 0, G, D, &a.n_splits, &a.span);
  a.max_len = max_len;
  a.scale = scale;
  a.k_pages = k_pages; a.v_pages = v_pages; a.logdeg_pages = logdeg_pages; a.page_shift = shift;
  a.k_new = k_new; a.v_new = v_new;
  a.k_pages_w = k_pages; a.v_pages_w = v_pages; a.deg_pages_w = deg_pages; a.logdeg_pages_w = logdeg_pages;
  return launch_decode_paged(a, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CKV_OK : CKV_ERR_CUDA;
}

}  // extern "C"
