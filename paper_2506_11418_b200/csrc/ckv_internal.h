// Internal interfaces between the host driver (ckv_api.cu) and the kernel files.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

namespace ckv {

enum RoundMode : int32_t {
  kModeAll = 0,       // every edge is merged (ratio 1)
  kModeChunkTopM = 1, // the best m edges of each chunk are merged
  kModeExternal = 2,  // edge targets, selection flags and output offsets come from global memory
  kModeMatchOnly = 3  // write each A token's edge (similarity, target) and stop
};

// One clustering round over the middle region [lo, hi) of every (layer, head) slab.
struct RoundArgs {
  const void* k_src;
  const void* v_src;
  const int32_t* deg_src;  // may be null: all ones
  void* k_dst;
  void* v_dst;
  int32_t* deg_dst;
  float* logdeg_dst;       // may be null
  int32_t* assign;         // may be null; [LH, assign_stride] slot of each source token, this round
  int64_t assign_stride;
  int64_t src_cap, dst_cap;
  int64_t lo, hi;
  int64_t out_lo;          // dst position of the first chunk's first survivor (kModeAll, kModeChunkTopM)
  int32_t chunk, n_chunks;  // chunk size; chunks per slab (the stride of the per-chunk arrays)
  int32_t chunk_first;      // this launch covers chunks [chunk_first, chunk_first + n_launch) of every slab
  int32_t n_launch;
  int32_t mode;
  int32_t m_full, m_tail;  // kModeChunkTopM: merges in a full chunk / in the shorter last chunk
  int64_t out_stride;      // kModeAll, kModeChunkTopM: survivors of a full chunk
  float* edge_sim;         // [LH, edge_stride]   kModeMatchOnly writes, select kernel reads
  int32_t* edge_b;         // [LH, edge_stride]   local offset of the edge's B token, -1 = no candidate
  uint8_t* sel;            // [LH, edge_stride]   kModeExternal: 1 = merge this edge
  int32_t* chunk_out_off;  // [LH, n_chunks]      kModeExternal: dst position of the chunk's first survivor
  int64_t edge_stride;     // n_chunks * chunk / 2
  int32_t LH;
  int32_t* status;         // device word in the workspace: nonzero after a bounded wait gave up
  int32_t overlap;         // 1: this launch depends on nothing the kernels since the last ordered launch write (see below)
};

// Copy `count` token rows (K, V, degree) of every slab from src_off to dst_off.
struct CopyArgs {
  const void* k_src;
  const void* v_src;
  const int32_t* deg_src;  // may be null: ones
  void* k_dst;
  void* v_dst;
  int32_t* deg_dst;
  float* logdeg_dst;       // may be null
  int32_t* assign;         // may be null
  int64_t assign_stride;
  int64_t src_cap, dst_cap, src_off, dst_off, count;
  int32_t LH;
  int32_t overlap;         // 1: see RoundArgs::overlap
};

// One new token (degree 1) for each of up to kAppendBatchMax sequences: token b of k_new / v_new [LH, n_total, D] goes
// to slot len[b] of sequence b.
constexpr int kAppendBatchMax = 64;
struct AppendBatchArgs {
  const void* k_new;
  const void* v_new;
  void* k[kAppendBatchMax];
  void* v[kAppendBatchMax];
  int32_t* deg[kAppendBatchMax];
  float* logdeg[kAppendBatchMax];  // entries may be null
  int64_t cap[kAppendBatchMax];
  int64_t len[kAppendBatchMax];
  int32_t n;        // sequences in this launch
  int32_t first;    // index of the first of them in k_new / v_new
  int32_t n_total;  // sequences in k_new / v_new
  int32_t LH;
};

// A cache in pages (the block layout of serving engines): per layer one pool k, v [n_pages, H, page_tokens, D], deg and
// logdeg [n_pages, H, page_tokens]; a sequence's token t sits in page table[t >> shift] at offset t & (page_tokens - 1).
// A round reads the sequence through src_table and writes it through dst_table (other pages of the same pools).
constexpr int kMaxPoolLayers = 64;
struct PagedArgs {
  unsigned char* k[kMaxPoolLayers];
  unsigned char* v[kMaxPoolLayers];
  int32_t* deg[kMaxPoolLayers];
  float* logdeg[kMaxPoolLayers];   // entries may be null
  const int32_t* src_table;
  const int32_t* dst_table;
  int64_t dst_last_page;           // last entry of dst_table that the round's output reaches
  int32_t H, shift;
};
struct NoPages {};

// Row copies between the two homes a sequence can have: pages of the per-layer pools, or a contiguous [LH, cap] slab.
struct RowsEnd {
  const int32_t* table;  // non-null: the rows live in pages (pools of the PagedArgs that comes with the call)
  unsigned char* k;      // else: slab arrays
  unsigned char* v;
  int32_t* deg;
  float* logdeg;         // may be null
  int64_t cap;
};
struct RowsCopyArgs {
  RowsEnd src, dst;
  int64_t src_off, dst_off, count;  // `count` rows from position src_off to position dst_off, for every slab
  // optional (device): for slab lh the copy starts at dst position begin[lh * begin_stride + begin_index] instead of
  // dst_off and ends at dst_end; the source moves along (src position = src_off + (position - dst_off))
  const int32_t* begin;
  int64_t begin_stride, begin_index, dst_end;
  int32_t LH, row_bytes;
  bool src_has_deg;  // else every copied row gets degree 1
};

struct SelectArgs {
  const float* edge_sim;
  uint8_t* sel;
  int32_t* chunk_out_off;
  int64_t edge_stride;
  int64_t M;       // edges to merge per (layer, head)
  int64_t lo;
  int32_t chunk, n_chunks;
  int32_t LH;
};

struct DecodeArgs {
  const void* views;  // const ckv_layer_view*, or const ckv_paged_view* when the cache is paged
  const void* q;
  void* out;
  float* partial;     // [Bz, H*G, n_splits, D + 4]: out[D], max, sum, pad
  int32_t Bz, H, G;
  int32_t n_splits;
  int64_t span;       // tokens per split
  int64_t max_len;    // longest sequence of the batch (host's bound; chooses the launch shape)
  float scale;
  // paged cache (bf16 kernel only): pages of `page_tokens` tokens, [n_pages, H, page_tokens, D]
  const void* k_pages;
  const void* v_pages;
  const float* logdeg_pages;  // [n_pages, H, page_tokens] or null
  int32_t page_shift;         // log2(page_tokens), page_tokens >= 32
  // paged, fused append (all null otherwise): sequence b's new token k_new / v_new [Bz, H, D] is attended to as
  // position len and written to that slot of its page with degree 1
  const void* k_new;
  const void* v_new;
  void* k_pages_w;
  void* v_pages_w;
  int32_t* deg_pages_w;
  float* logdeg_pages_w;      // may be null
};

// Streaming multiprocessors of the current device, asked once per device (the grids are sized from it).
inline int sm_count() {
  constexpr int kMaxDev = 64;
  static std::atomic<int> cached[kMaxDev];
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  const bool slot = dev >= 0 && dev < kMaxDev;
  if (slot && (n = cached[dev].load(std::memory_order_relaxed)) > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  if (slot) cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

// Launch with programmatic stream serialization: the kernel may become resident while the kernel ahead of it
// in the stream drains; it must call griddep_wait() before it touches anything that kernel produced.
//
// How the kernels of a clustering round use it.  An ORDERED kernel calls griddep_wait() and then griddep_launch() before
// anything else: it starts after everything ahead of it has completed, and lets the next launch become resident as its
// own CTAs leave.  A kernel launched with `overlap` = 1 (the shorter last chunk of a pass, the copies of sinks and recent
// tokens) skips the wait at its start and calls griddep_wait() as its last statement instead: it runs beside the ordered
// kernel ahead of it and beside other overlap launches in between, so it may neither read what those write nor write
// what they read; because it cannot complete before its predecessor has, "the kernel ahead has completed" still means
// "everything before it has completed" for whatever comes next.  The host sets overlap only after an ordered kernel
// of the same round has been launched.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

cudaError_t launch_round(const RoundArgs& a, int dtype, int D, cudaStream_t st);
cudaError_t launch_copy(const CopyArgs& a, int dtype, int D, cudaStream_t st);
cudaError_t launch_select(const SelectArgs& a, cudaStream_t st);
int page_shift(int32_t page_tokens);  // log2 of a valid page size (a power of two >= 32), else -1
cudaError_t launch_rows_copy(const RowsCopyArgs& a, const PagedArgs& pools, cudaStream_t st);
cudaError_t launch_append_batch(const AppendBatchArgs& a, int dtype, int D, cudaStream_t st);
cudaError_t launch_compose_assign(int32_t* total, const int32_t* step, int64_t n_src, int64_t step_stride, int32_t LH,
                                  cudaStream_t st);
cudaError_t launch_decode(const DecodeArgs& a, int dtype, int D, cudaStream_t st);
cudaError_t launch_decode_paged(const DecodeArgs& a, cudaStream_t st);
void decode_plan(int32_t Bz, int32_t H, int dtype, int64_t max_len, int64_t max_partial_floats, int32_t G, int32_t D,
                 int32_t* n_splits, int64_t* span);
size_t decode_partial_floats(int32_t Bz, int32_t H, int32_t G, int32_t D, int64_t max_len);
size_t round_smem_bytes(int chunk, int D);
bool round_fast_supported(const RoundArgs& a, int dtype, int D);
cudaError_t launch_round_fast(const RoundArgs& a, int64_t n_full, cudaStream_t st);
// the same round on a paged cache (a.k_src, a.k_dst ... are not used; a.deg_src != null only says that the pages carry degrees)
cudaError_t launch_round_fast_paged(const RoundArgs& a, const PagedArgs& pg, int64_t n_full, cudaStream_t st);
bool round_umma_supported(const RoundArgs& a, int dtype, int D);
cudaError_t launch_round_umma(const RoundArgs& a, int64_t n_full, cudaStream_t st);
bool bsm_supported(int dtype, int D);
size_t bsm_workspace_bytes(int64_t LH, int64_t mid);
cudaError_t launch_bsm_match(const RoundArgs& a, void* scratch, cudaStream_t st);  // a.lo, a.hi: the middle region
cudaError_t launch_bsm_merge(const RoundArgs& a, void* scratch, cudaStream_t st);
// two consecutive ratio-1 rounds at chunk 64 in one pass (source degrees all one): rounds j, j + 1 on the first
// 2 * units chunks of every slab; assign2 / stride2: the second round's slot map when a.assign is given
bool round_fused2_supported(int dtype, int D, int chunk);
cudaError_t launch_round_fused2(const RoundArgs& a, int64_t units, int32_t* assign2, int64_t stride2, cudaStream_t st);
// chunk 128 / 256 in the modes that merge: groups of warps per chunk, warp-level tensor-core matching and merge
bool round_group_supported(const RoundArgs& a, int dtype, int D);
cudaError_t launch_round_group(const RoundArgs& a, int64_t n_full, cudaStream_t st);
bool round_tile_supported(const RoundArgs& a, int dtype, int D);
cudaError_t launch_round_tile(const RoundArgs& a, cudaStream_t st);

}  // namespace ckv
