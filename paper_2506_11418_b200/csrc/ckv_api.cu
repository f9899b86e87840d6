// Host side of the C ABI: argument checks, the round schedule of Algorithm 1 / Eq. 4, workspace
// layout, and the launch sequences.  No device memory is allocated here.
#include <cmath>
#include <utility>
#include <cstring>
#include <vector>

#include "../../include/ckv.h"
#include "ckv_internal.h"

namespace ckv {
namespace {

struct RoundPlan {
  int64_t s_in, s_out, lo, hi;
  int32_t n_chunks;
  int64_t n_edges;  // A tokens that have a B candidate
  int64_t M;        // merges per (layer, head)
  int32_t m_full, m_tail;
  int32_t mode;     // RoundMode, or -1: nothing merges (verbatim copy)
};

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

int check_params(const ckv_params* p) {
  if (!p) return CKV_ERR_INVALID_ARG;
  if (p->chunk != 0 && (p->chunk < 2 || (p->chunk & 1))) return CKV_ERR_INVALID_ARG;  // 0: no chunking
  if (p->n_sink < 0 || p->n_recent < 0 || p->n_rounds_max < 0 || p->budget < 0) return CKV_ERR_INVALID_ARG;
  if (!(p->r_init >= 0.f && p->r_init <= 1.f) || !(p->r_decay >= 0.f) || !(p->r_min >= 0.f && p->r_min <= 1.f))
    return CKV_ERR_INVALID_ARG;
  if (p->select != CKV_SELECT_GLOBAL && p->select != CKV_SELECT_CHUNK) return CKV_ERR_INVALID_ARG;
  if (p->chunk > 256) return CKV_ERR_UNSUPPORTED;
  return CKV_OK;
}

inline int64_t floor_ratio(double r, int64_t n) { return (int64_t)std::floor(r * (double)n + 1e-9); }

// Algorithm 1's `while s > B` loop with Eq. 4: everything a round does is a function of lengths.
int plan_rounds(int64_t len, const ckv_params& p, std::vector<RoundPlan>& plan) {
  plan.clear();
  int64_t s = len;
  for (int j = 0; j < p.n_rounds_max && (p.budget == 0 || s > p.budget); ++j) {
    const double r = std::fmax((double)p.r_init - (double)j * (double)p.r_decay, (double)p.r_min);
    RoundPlan rp{};
    rp.s_in = s;
    rp.lo = std::min<int64_t>(p.n_sink, s);
    rp.hi = std::max<int64_t>(rp.lo, s - p.n_recent);
    const int64_t mid = rp.hi - rp.lo;
    if (p.chunk == 0) {
      // no chunking (plain Bipartite Soft Matching): the middle region is one chunk; ranking per chunk and per head coincide
      rp.n_chunks = mid >= 2 ? 1 : 0;
      rp.n_edges = mid >= 2 ? (mid + 1) / 2 : 0;
      rp.M = floor_ratio(r, rp.n_edges);
      if (p.budget > 0 && p.select == CKV_SELECT_GLOBAL) rp.M = std::min<int64_t>(rp.M, s - p.budget);
      rp.mode = rp.M == 0 ? -1 : kModeExternal;
      rp.m_full = rp.m_tail = 0;
      rp.s_out = s - rp.M;
      if (rp.M == 0 && p.budget > 0) return CKV_ERR_NO_PROGRESS;
      plan.push_back(rp);
      s = rp.s_out;
      continue;
    }
    const int c = p.chunk;
    const int64_t n_full = mid >= 2 ? mid / c : 0;
    const int tail = mid >= 2 ? (int)(mid % c) : 0;
    rp.n_chunks = (int32_t)(n_full + (tail > 0 ? 1 : 0));
    const int64_t tail_edges = tail >= 2 ? (tail + 1) / 2 : 0;
    rp.n_edges = n_full * (c / 2) + tail_edges;
    if (p.select == CKV_SELECT_GLOBAL) {
      rp.M = floor_ratio(r, rp.n_edges);
      if (p.budget > 0) rp.M = std::min<int64_t>(rp.M, s - p.budget);
      rp.mode = rp.M == 0 ? -1 : (rp.M == rp.n_edges ? kModeAll : kModeExternal);
      rp.m_full = c / 2;
      rp.m_tail = (int32_t)tail_edges;
    } else {
      rp.m_full = (int32_t)floor_ratio(r, c / 2);
      rp.m_tail = (int32_t)floor_ratio(r, tail_edges);
      rp.M = n_full * rp.m_full + rp.m_tail;
      rp.mode = rp.M == 0 ? -1 : ((rp.m_full == c / 2 && rp.m_tail == tail_edges) ? kModeAll : kModeChunkTopM);
    }
    rp.s_out = s - rp.M;
    if (rp.M == 0 && p.budget > 0) return CKV_ERR_NO_PROGRESS;
    plan.push_back(rp);
    s = rp.s_out;
  }
  return CKV_OK;
}

// Which buffer each round writes: the last one lands in dst, the others alternate with tmp.
inline bool round_targets_dst(size_t j, size_t R) { return ((R - 1 - j) & 1) == 0; }

struct Workspace {
  size_t tmp_k, tmp_v, tmp_deg, tmp_logdeg;  // offsets; tmp cache [LH, tmp_cap, D]
  int64_t tmp_cap;
  size_t edge_sim, edge_b, sel, chunk_off;
  int64_t edge_stride;
  size_t bsm;  // scratch of the no-chunk rounds
  size_t assign_step;
  int64_t assign_stride;
  size_t total;
};

Workspace layout_workspace(int64_t LH, int D, int esize, int chunk, const std::vector<RoundPlan>& plan,
                           bool want_assign) {
  Workspace w{};
  const size_t R = plan.size();
  int64_t max_chunks = 0, max_sin = 0;
  for (size_t j = 0; j < R; ++j) {
    if (!round_targets_dst(j, R)) w.tmp_cap = std::max(w.tmp_cap, plan[j].s_out);
    if (plan[j].mode == kModeExternal) max_chunks = std::max<int64_t>(max_chunks, plan[j].n_chunks);
    max_sin = std::max(max_sin, plan[j].s_in);
  }
  size_t off = 256;  // the first 256 bytes hold the device status word
  auto take = [&off](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes);
    return at;
  };
  w.tmp_k = take((size_t)LH * w.tmp_cap * D * esize);
  w.tmp_v = take((size_t)LH * w.tmp_cap * D * esize);
  w.tmp_deg = take((size_t)LH * w.tmp_cap * 4);
  w.tmp_logdeg = take((size_t)LH * w.tmp_cap * 4);
  w.edge_stride = max_chunks * (chunk / 2);
  int64_t bsm_mid = 0;
  if (chunk == 0)
    for (size_t j = 0; j < R; ++j) {
      w.edge_stride = std::max(w.edge_stride, plan[j].n_edges);
      bsm_mid = std::max(bsm_mid, plan[j].hi - plan[j].lo);
    }
  w.edge_sim = take((size_t)LH * w.edge_stride * 4);
  w.edge_b = take((size_t)LH * w.edge_stride * 4);
  w.sel = take((size_t)LH * w.edge_stride);
  w.chunk_off = take((size_t)LH * std::max<int64_t>(max_chunks, 1) * 4);
  w.bsm = take(chunk == 0 ? bsm_workspace_bytes(LH, bsm_mid) : 0);
  w.assign_stride = (want_assign && R >= 2) ? max_sin : 0;
  w.assign_step = take((size_t)LH * w.assign_stride * 4);
  w.total = off;
  return w;
}

inline int esize_of(int dtype) { return dtype == CKV_F32 ? 4 : 2; }

int check_cache_shape(const ckv_cache* c, bool with_len = true) {
  if (!c) return CKV_ERR_INVALID_ARG;
  if (c->L <= 0 || c->H <= 0 || c->D <= 0 || c->cap < 0) return CKV_ERR_INVALID_ARG;
  if (with_len && (c->len < 0 || c->len > c->cap || c->pending < 0 || c->pending > c->len)) return CKV_ERR_INVALID_ARG;
  if (c->dtype != CKV_F32 && c->dtype != CKV_BF16) return CKV_ERR_INVALID_ARG;
  if ((int64_t)c->L * c->H > 65535) return CKV_ERR_UNSUPPORTED;
  if (c->D != 128) return CKV_ERR_UNSUPPORTED;
  return CKV_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline bool overlaps(const void* a, size_t an, const void* b, size_t bn) {
  const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
  return an && bn && x < y + bn && y < x + an;
}

struct Buf {  // one cache buffer a round reads or writes
  void* k;
  void* v;
  int32_t* deg;
  float* logdeg;
  int64_t cap;
};

// One clustering round src -> dst (Sec. 5.2, Sec. 5.3, Eq. 5), sinks and recent tokens copied verbatim.
// first_chunk > 0 (chunked rounds that merge every edge only): the chunks before it are someone else's work.
cudaError_t run_round(const RoundPlan& rp, const Buf& src, const Buf& dst, int LH, int D, int dtype, int chunk,
                      int32_t* assign, int64_t assign_stride, const Workspace& w, unsigned char* ws, cudaStream_t st,
                      int32_t first_chunk = 0) {
  cudaError_t e;
  CopyArgs c{};
  c.k_src = src.k; c.v_src = src.v; c.deg_src = src.deg;
  c.k_dst = dst.k; c.v_dst = dst.v; c.deg_dst = dst.deg; c.logdeg_dst = dst.logdeg;
  c.assign = assign; c.assign_stride = assign_stride;
  c.src_cap = src.cap; c.dst_cap = dst.cap; c.LH = LH;
  if (rp.mode < 0) {  // nothing merges: the round is the identity
    c.src_off = 0; c.dst_off = 0; c.count = rp.s_in;
    return launch_copy(c, dtype, D, st);
  }
  // Sinks and recent tokens.  After an ordered kernel of this round they may run beside the kernels of the round (they
  // touch rows no chunk owns, and every earlier round has completed by then); on their own they are ordered launches.
  auto copy_edges = [&](bool beside) -> cudaError_t {
    c.overlap = beside ? 1 : 0;
    c.src_off = 0; c.dst_off = 0; c.count = rp.lo;
    cudaError_t ce = launch_copy(c, dtype, D, st);
    if (ce != cudaSuccess) return ce;
    c.src_off = rp.hi; c.dst_off = rp.hi - rp.M; c.count = rp.s_in - rp.hi;
    return launch_copy(c, dtype, D, st);
  };
  if (chunk == 0 && (e = copy_edges(false)) != cudaSuccess) return e;

  RoundArgs a{};
  a.k_src = src.k; a.v_src = src.v; a.deg_src = src.deg;
  a.k_dst = dst.k; a.v_dst = dst.v; a.deg_dst = dst.deg; a.logdeg_dst = dst.logdeg;
  a.assign = assign; a.assign_stride = assign_stride;
  a.src_cap = src.cap; a.dst_cap = dst.cap;
  a.lo = rp.lo; a.hi = rp.hi;
  if (chunk == 0) {
    // no chunking: norms + tensor-core matching over all A x B pairs of a head, ranking, merge by member scan
    if (!bsm_supported(dtype, D)) return cudaErrorInvalidValue;
    a.LH = LH;
    a.status = reinterpret_cast<int32_t*>(ws);
    a.edge_stride = rp.n_edges;
    a.edge_sim = reinterpret_cast<float*>(ws + w.edge_sim);
    a.edge_b = reinterpret_cast<int32_t*>(ws + w.edge_b);
    a.sel = ws + w.sel;
    a.chunk_out_off = reinterpret_cast<int32_t*>(ws + w.chunk_off);
    if ((e = launch_bsm_match(a, ws + w.bsm, st)) != cudaSuccess) return e;
    SelectArgs s{};
    s.edge_sim = a.edge_sim; s.sel = a.sel; s.chunk_out_off = a.chunk_out_off;
    s.edge_stride = a.edge_stride; s.M = rp.M; s.lo = rp.lo; s.chunk = (int32_t)(2 * rp.n_edges); s.n_chunks = 1; s.LH = LH;
    if ((e = launch_select(s, st)) != cudaSuccess) return e;
    return launch_bsm_merge(a, ws + w.bsm, st);
  }
  a.chunk = chunk; a.n_chunks = rp.n_chunks;
  a.chunk_first = first_chunk; a.n_launch = rp.n_chunks - first_chunk;
  if (a.n_launch <= 0) return copy_edges(false);
  a.m_full = rp.m_full; a.m_tail = rp.m_tail;
  a.out_stride = chunk - rp.m_full;
  a.out_lo = rp.lo;
  a.LH = LH;
  a.status = reinterpret_cast<int32_t*>(ws);
  a.edge_stride = (int64_t)rp.n_chunks * (chunk / 2);
  // bf16: the full chunks of chunk 64 go to the warp-per-chunk kernel, those of chunk 256 to the tcgen05 kernel, chunk 128
  // and every shorter last chunk to the tile kernel; everything else runs on the general kernel
  auto launch_pass = [&](RoundArgs x) -> cudaError_t {
    const bool fast = round_fast_supported(x, dtype, D), group = !fast && round_group_supported(x, dtype, D);
    const bool umma = !fast && !group && round_umma_supported(x, dtype, D);
    if (fast || group || umma) {
      const int64_t n_full = (rp.hi - rp.lo) / chunk;
      if (!fast && first_chunk > 0) return cudaErrorInvalidValue;
      if (n_full > first_chunk) {
        cudaError_t err = fast ? launch_round_fast(x, n_full, st) : (group ? launch_round_group(x, n_full, st) : launch_round_umma(x, n_full, st));
        if (err != cudaSuccess) return err;
        x.overlap = 1;  // the shorter last chunk is nobody else's: it may run beside the full chunks just launched
      }
      if (rp.n_chunks == n_full) return cudaSuccess;
      x.chunk_first = (int32_t)std::max<int64_t>(n_full, first_chunk);
      x.n_launch = rp.n_chunks - x.chunk_first;
    }
    return round_tile_supported(x, dtype, D) ? launch_round_tile(x, st) : launch_round(x, dtype, D, st);
  };
  if (rp.mode == kModeExternal) {
    a.edge_sim = reinterpret_cast<float*>(ws + w.edge_sim);
    a.edge_b = reinterpret_cast<int32_t*>(ws + w.edge_b);
    a.sel = ws + w.sel;
    a.chunk_out_off = reinterpret_cast<int32_t*>(ws + w.chunk_off);
    a.mode = kModeMatchOnly;
    if ((e = launch_pass(a)) != cudaSuccess) return e;
    SelectArgs s{};
    s.edge_sim = a.edge_sim; s.sel = a.sel; s.chunk_out_off = a.chunk_out_off;
    s.edge_stride = a.edge_stride; s.M = rp.M; s.lo = rp.lo; s.chunk = chunk; s.n_chunks = rp.n_chunks; s.LH = LH;
    if ((e = launch_select(s, st)) != cudaSuccess) return e;
  }
  a.mode = rp.mode;
  if ((e = launch_pass(a)) != cudaSuccess) return e;
  return copy_edges(true);  // (the pass above began with an ordered launch)
}

// Runs the planned rounds from `src` into `dst` (ping-pong through the workspace's tmp cache).
int run_plan(const std::vector<RoundPlan>& plan, const Buf& src, const Buf& dst, int64_t src_len, int LH, int D,
             int dtype, int chunk, int32_t* assign, Workspace& w, unsigned char* ws, cudaStream_t st) {
  const size_t R = plan.size();
  cudaError_t e;
  if (R == 0) {
    RoundPlan id{};
    id.s_in = src_len;
    id.mode = -1;
    e = run_round(id, src, dst, LH, D, dtype, chunk, assign, src_len, w, ws, st);
    return e == cudaSuccess ? CKV_OK : CKV_ERR_CUDA;
  }
  Buf tmp{ws + w.tmp_k, ws + w.tmp_v, reinterpret_cast<int32_t*>(ws + w.tmp_deg),
          reinterpret_cast<float*>(ws + w.tmp_logdeg), w.tmp_cap};
  Buf cur = src;
  for (size_t j = 0; j < R; ++j) {
    // Two rounds in one pass: rounds j and j + 1 both merge every edge at chunk 64 and the source degrees are all
    // one.  Pairs of full round-1 chunks are exactly the full round-2 chunks they feed; those go through the fused
    // kernel straight into the second round's target.  What is left (an odd chunk, the shorter last chunk, sinks and
    // recent tokens) takes the two rounds one after the other.
    if (j + 1 < R && cur.deg == nullptr && plan[j].mode == kModeAll && plan[j + 1].mode == kModeAll &&
        plan[j].lo == plan[j + 1].lo && round_fused2_supported(dtype, D, chunk)) {
      const int64_t units = (plan[j].hi - plan[j].lo) / chunk / 2;
      if (units > 0) {
        const Buf& t1 = round_targets_dst(j, R) ? dst : tmp;
        const Buf& t2 = round_targets_dst(j + 1, R) ? dst : tmp;
        int32_t* step2 = assign ? reinterpret_cast<int32_t*>(ws + w.assign_step) : nullptr;
        RoundArgs f{};
        f.k_src = cur.k; f.v_src = cur.v;
        f.k_dst = t2.k; f.v_dst = t2.v; f.deg_dst = t2.deg; f.logdeg_dst = t2.logdeg;
        f.assign = assign; f.assign_stride = src_len;  // j == 0 here: only the caller's source has no degrees
        f.src_cap = cur.cap; f.dst_cap = t2.cap;
        f.lo = plan[j].lo; f.LH = LH;
        f.status = reinterpret_cast<int32_t*>(ws);
        if (launch_round_fused2(f, units, step2, w.assign_stride, st) != cudaSuccess) return CKV_ERR_CUDA;
        e = run_round(plan[j], cur, t1, LH, D, dtype, chunk, assign, src_len, w, ws, st, (int32_t)(2 * units));
        if (e != cudaSuccess) return CKV_ERR_CUDA;
        e = run_round(plan[j + 1], t1, t2, LH, D, dtype, chunk, step2, w.assign_stride, w, ws, st, (int32_t)units);
        if (e != cudaSuccess) return CKV_ERR_CUDA;
        if (assign && launch_compose_assign(assign, step2, src_len, w.assign_stride, LH, st) != cudaSuccess) return CKV_ERR_CUDA;
        cur = t2;
        ++j;
        continue;
      }
    }
    const Buf& target = round_targets_dst(j, R) ? dst : tmp;
    int32_t* step = nullptr;
    int64_t step_stride = 0;
    if (assign) {
      if (j == 0) {
        step = assign;
        step_stride = src_len;
      } else {
        step = reinterpret_cast<int32_t*>(ws + w.assign_step);
        step_stride = w.assign_stride;
      }
    }
    e = run_round(plan[j], cur, target, LH, D, dtype, chunk, step, step_stride, w, ws, st);
    if (e != cudaSuccess) return CKV_ERR_CUDA;
    if (assign && j > 0) {
      e = launch_compose_assign(assign, step, src_len, step_stride, LH, st);
      if (e != cudaSuccess) return CKV_ERR_CUDA;
    }
    cur = target;
  }
  return CKV_OK;
}

// Capacity dst needs: everything a round writes into it.
int64_t dst_cap_needed(const std::vector<RoundPlan>& plan, int64_t len) {
  const size_t R = plan.size();
  if (R == 0) return len;
  int64_t need = 0;
  for (size_t j = 0; j < R; ++j)
    if (round_targets_dst(j, R)) need = std::max(need, plan[j].s_out);
  return need;
}

// A completed window of `c` appended tokens at the tail of the cache is clustered on its own: copied aside, then the
// planned rounds run back into its place.  cache->len is updated.
int cluster_window(ckv_cache* cache, const std::vector<RoundPlan>& plan, int64_t win_out, int64_t LH, int D, int es, int c,
                   Workspace& w, unsigned char* ws, const Buf& stage, cudaStream_t stream) {
  const int64_t w0 = cache->len - c;
  CopyArgs out{};
  out.k_src = cache->k; out.v_src = cache->v; out.deg_src = cache->deg;
  out.k_dst = stage.k; out.v_dst = stage.v; out.deg_dst = stage.deg; out.logdeg_dst = stage.logdeg;
  out.src_cap = cache->cap; out.dst_cap = c; out.src_off = w0; out.dst_off = 0; out.count = c; out.LH = (int)LH;
  if (launch_copy(out, cache->dtype, D, stream) != cudaSuccess) return CKV_ERR_CUDA;
  // the window's destination is a view of the cache that starts at w0
  const Buf dstw{static_cast<unsigned char*>(cache->k) + (size_t)w0 * D * es,
                 static_cast<unsigned char*>(cache->v) + (size_t)w0 * D * es, cache->deg + w0,
                 cache->logdeg ? cache->logdeg + w0 : nullptr, cache->cap};
  const int st = run_plan(plan, stage, dstw, c, (int)LH, D, cache->dtype, c, nullptr, w, ws, stream);
  if (st != CKV_OK) return st;
  cache->len = w0 + win_out;
  return CKV_OK;
}

ckv_params window_params(const ckv_params& p) {
  ckv_params wp = p;
  wp.n_sink = 0;
  wp.n_recent = 0;
  return wp;
}

// ---- clustering a paged cache in place of a slab (bf16, chunk 64) ---------------------------------------------------
// The full chunks go through the warp-per-chunk kernel, which fetches a chunk's rows from its page (two pieces when the
// chunk straddles a page boundary) and writes the surviving rows into the destination pages.  The shorter last chunk of
// a round is staged: its rows are copied to a small slab, the tile kernel clusters it slab to slab, and the result is
// copied into the destination pages.  Sinks and recent tokens are row copies from pages to pages.

struct PagedWorkspace {
  size_t edge_sim, edge_b, sel, chunk_off;
  int64_t edge_stride, max_chunks;
  size_t a_k, a_v, a_deg, b_k, b_v, b_deg, b_logdeg;  // staging slabs [LH, 64, ...] of the last chunk
  size_t total;
};

PagedWorkspace layout_paged_workspace(int64_t LH, int D, int es, int chunk, const std::vector<RoundPlan>& plan) {
  PagedWorkspace w{};
  for (const RoundPlan& rp : plan)
    if (rp.mode == kModeExternal) w.max_chunks = std::max<int64_t>(w.max_chunks, rp.n_chunks);
  size_t off = 256;
  auto take = [&off](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes);
    return at;
  };
  w.edge_stride = w.max_chunks * (chunk / 2);
  w.edge_sim = take((size_t)LH * w.edge_stride * 4);
  w.edge_b = take((size_t)LH * w.edge_stride * 4);
  w.sel = take((size_t)LH * w.edge_stride);
  w.chunk_off = take((size_t)LH * std::max<int64_t>(w.max_chunks, 1) * 4);
  const size_t kv = (size_t)LH * chunk * D * es, dg = (size_t)LH * chunk * 4;
  w.a_k = take(kv); w.a_v = take(kv); w.a_deg = take(dg);
  w.b_k = take(kv); w.b_v = take(kv); w.b_deg = take(dg); w.b_logdeg = take(dg);
  w.total = off;
  return w;
}

cudaError_t run_round_paged(const RoundPlan& rp, PagedArgs pg, bool src_has_deg, int LH, int D, int chunk, const PagedWorkspace& w,
                            unsigned char* ws, cudaStream_t st) {
  cudaError_t e;
  const int es = 2, row_bytes = D * es;
  pg.dst_last_page = std::max<int64_t>(rp.s_out - 1, 0) >> pg.shift;
  RowsCopyArgs c{};
  c.src.table = pg.src_table; c.dst.table = pg.dst_table;
  c.LH = LH; c.row_bytes = row_bytes; c.src_has_deg = src_has_deg;
  if (rp.mode < 0) {  // nothing merges: the round is the identity
    c.src_off = 0; c.dst_off = 0; c.count = rp.s_in;
    return launch_rows_copy(c, pg, st);
  }
  c.src_off = 0; c.dst_off = 0; c.count = rp.lo;
  if ((e = launch_rows_copy(c, pg, st)) != cudaSuccess) return e;
  c.src_off = rp.hi; c.dst_off = rp.hi - rp.M; c.count = rp.s_in - rp.hi;
  if ((e = launch_rows_copy(c, pg, st)) != cudaSuccess) return e;

  const int64_t n_full = (rp.hi - rp.lo) / chunk;
  const bool has_tail = rp.n_chunks > n_full;
  const int64_t p_tail = rp.lo + n_full * chunk, tail = rp.hi - p_tail;
  const int64_t q_end = rp.hi - rp.M;  // where the middle region's output ends
  RoundArgs a{};
  a.deg_src = src_has_deg ? reinterpret_cast<const int32_t*>(ws) : nullptr;  // only says: the pages carry degrees
  a.lo = rp.lo; a.hi = rp.hi;
  a.chunk = chunk; a.n_chunks = rp.n_chunks;
  a.m_full = rp.m_full; a.m_tail = rp.m_tail;
  a.out_stride = chunk - rp.m_full;
  a.out_lo = rp.lo;
  a.LH = LH;
  a.status = reinterpret_cast<int32_t*>(ws);
  a.edge_stride = (int64_t)rp.n_chunks * (chunk / 2);
  // the last chunk as a slab-to-slab round: base pointers shifted so that the chunk's positions in the sequence (source
  // p_tail ..., output ... q_end) index rows 0 .. 63 of the staging slabs
  RoundArgs t = a;
  const int64_t vbase = q_end - chunk;
  t.k_src = ws + w.a_k - p_tail * row_bytes; t.v_src = ws + w.a_v - p_tail * row_bytes;
  t.deg_src = src_has_deg ? reinterpret_cast<const int32_t*>(ws + w.a_deg) - p_tail : nullptr;
  t.k_dst = ws + w.b_k - vbase * row_bytes; t.v_dst = ws + w.b_v - vbase * row_bytes;
  t.deg_dst = reinterpret_cast<int32_t*>(ws + w.b_deg) - vbase;
  t.logdeg_dst = reinterpret_cast<float*>(ws + w.b_logdeg) - vbase;
  t.src_cap = chunk; t.dst_cap = chunk;
  t.chunk_first = (int32_t)n_full; t.n_launch = 1;
  if (has_tail) {
    RowsCopyArgs in{};
    in.src.table = pg.src_table;
    in.dst.k = ws + w.a_k; in.dst.v = ws + w.a_v; in.dst.deg = reinterpret_cast<int32_t*>(ws + w.a_deg); in.dst.cap = chunk;
    in.src_off = p_tail; in.dst_off = 0; in.count = tail;
    in.LH = LH; in.row_bytes = row_bytes; in.src_has_deg = src_has_deg;
    if ((e = launch_rows_copy(in, pg, st)) != cudaSuccess) return e;
  }
  auto launch_pass = [&](int mode) -> cudaError_t {
    RoundArgs x = a;
    x.mode = mode;
    cudaError_t err = launch_round_fast_paged(x, pg, n_full, st);
    if (err != cudaSuccess || !has_tail) return err;
    RoundArgs y = t;
    y.mode = mode;
    y.edge_sim = x.edge_sim; y.edge_b = x.edge_b; y.sel = x.sel; y.chunk_out_off = x.chunk_out_off;
    return launch_round_tile(y, st);
  };
  if (rp.mode == kModeExternal) {
    a.edge_sim = reinterpret_cast<float*>(ws + w.edge_sim);
    a.edge_b = reinterpret_cast<int32_t*>(ws + w.edge_b);
    a.sel = ws + w.sel;
    a.chunk_out_off = reinterpret_cast<int32_t*>(ws + w.chunk_off);
    if ((e = launch_pass(kModeMatchOnly)) != cudaSuccess) return e;
    SelectArgs sa{};
    sa.edge_sim = a.edge_sim; sa.sel = a.sel; sa.chunk_out_off = a.chunk_out_off;
    sa.edge_stride = a.edge_stride; sa.M = rp.M; sa.lo = rp.lo; sa.chunk = chunk; sa.n_chunks = rp.n_chunks; sa.LH = LH;
    if ((e = launch_select(sa, st)) != cudaSuccess) return e;
  }
  if ((e = launch_pass(rp.mode)) != cudaSuccess) return e;
  if (has_tail) {
    RowsCopyArgs out{};
    out.src.k = ws + w.b_k; out.src.v = ws + w.b_v; out.src.deg = reinterpret_cast<int32_t*>(ws + w.b_deg); out.src.cap = chunk;
    out.dst.table = pg.dst_table;
    out.LH = LH; out.row_bytes = row_bytes; out.src_has_deg = true;
    out.dst_end = q_end;
    if (rp.mode == kModeExternal) {  // where the last chunk's survivors start is only known on the device
      out.begin = a.chunk_out_off; out.begin_stride = rp.n_chunks; out.begin_index = n_full;
      out.src_off = 0; out.dst_off = vbase;
    } else {
      const int64_t q_tail = rp.lo + n_full * a.out_stride;
      out.src_off = q_tail - vbase; out.dst_off = q_tail; out.count = q_end - q_tail;
    }
    if ((e = launch_rows_copy(out, pg, st)) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

int paged_args_ok(const ckv_page_pool* pools, int32_t L, int32_t H, int32_t D, int32_t dtype, int32_t page_tokens,
                  const ckv_params* params) {
  int st;
  if ((st = check_params(params)) != CKV_OK) return st;
  if (!pools || L <= 0 || H <= 0) return CKV_ERR_INVALID_ARG;
  if (dtype != CKV_F32 && dtype != CKV_BF16) return CKV_ERR_INVALID_ARG;
  if (page_shift(page_tokens) < 0 || page_tokens < 64 || D != 128 || dtype != CKV_BF16 || params->chunk != 64 || L > kMaxPoolLayers ||
      (int64_t)L * H > 65535)
    return CKV_ERR_UNSUPPORTED;
  return CKV_OK;
}

}  // namespace
}  // namespace ckv

using namespace ckv;

extern "C" {

int ckv_pages_plan(int64_t len, const ckv_params* params, int32_t page_tokens, int64_t* out_len, int64_t* rounds,
                   int64_t* scratch_pages, int32_t* result_in_scratch, int64_t* pages_kept) {
  int st = check_params(params);
  if (st != CKV_OK) return st;
  if (len < 0 || page_tokens <= 0) return CKV_ERR_INVALID_ARG;
  std::vector<RoundPlan> plan;
  if ((st = plan_rounds(len, *params, plan)) != CKV_OK) return st;
  int64_t need = 0;
  for (size_t j = 0; j < plan.size(); j += 2) need = std::max(need, (plan[j].s_out + page_tokens - 1) / page_tokens);  // rounds 0, 2, ... land in the scratch pages
  const int64_t final_len = plan.empty() ? len : plan.back().s_out;
  if (out_len) *out_len = final_len;
  if (rounds) *rounds = (int64_t)plan.size();
  if (scratch_pages) *scratch_pages = need;
  if (result_in_scratch) *result_in_scratch = (int32_t)(plan.size() & 1);
  if (pages_kept) *pages_kept = (final_len + page_tokens - 1) / page_tokens;
  return CKV_OK;
}

size_t ckv_paged_workspace_bytes(int32_t L, int32_t H, int32_t D, int32_t dtype, int64_t len, const ckv_params* params) {
  if (check_params(params) != CKV_OK || L <= 0 || H <= 0 || len < 0 || params->chunk != 64) return 0;
  std::vector<RoundPlan> plan;
  if (plan_rounds(len, *params, plan) != CKV_OK) return 256;
  return layout_paged_workspace((int64_t)L * H, D, esize_of(dtype), params->chunk, plan).total;
}

int ckv_compress_paged(const ckv_page_pool* pools, int32_t L, int32_t H, int32_t D, int32_t dtype, int32_t page_tokens,
                       const int32_t* block_table, int64_t len, int32_t has_deg, const int32_t* scratch_table,
                       int64_t scratch_pages, const ckv_params* params, void* workspace, size_t workspace_bytes,
                       void* cuda_stream, int64_t* out_len, int32_t* result_in_scratch) {
  int st;
  if ((st = paged_args_ok(pools, L, H, D, dtype, page_tokens, params)) != CKV_OK) return st;
  if (!block_table || len < 0) return CKV_ERR_INVALID_ARG;
  PagedArgs pg{};
  for (int32_t l = 0; l < L; ++l) {
    if (!pools[l].k_pages || !pools[l].v_pages || !pools[l].deg_pages) return CKV_ERR_INVALID_ARG;
    if (!aligned16(pools[l].k_pages) || !aligned16(pools[l].v_pages)) return CKV_ERR_ALIGNMENT;
    pg.k[l] = static_cast<unsigned char*>(pools[l].k_pages);
    pg.v[l] = static_cast<unsigned char*>(pools[l].v_pages);
    pg.deg[l] = pools[l].deg_pages;
    pg.logdeg[l] = pools[l].logdeg_pages;
  }
  pg.H = H;
  pg.shift = page_shift(page_tokens);
  std::vector<RoundPlan> plan;
  if ((st = plan_rounds(len, *params, plan)) != CKV_OK) return st;
  int64_t need = 0;
  for (size_t j = 0; j < plan.size(); j += 2) need = std::max(need, (plan[j].s_out + page_tokens - 1) / page_tokens);
  if (need > 0 && (!scratch_table || scratch_pages < need)) return CKV_ERR_CAPACITY;
  const int64_t LH = (int64_t)L * H;
  const PagedWorkspace w = layout_paged_workspace(LH, D, esize_of(dtype), params->chunk, plan);
  if (!workspace || workspace_bytes < w.total || !aligned16(workspace)) return CKV_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, 256, stream) != cudaSuccess) return CKV_ERR_CUDA;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  bool src_has_deg = has_deg != 0;
  for (size_t j = 0; j < plan.size(); ++j) {
    pg.src_table = (j & 1) ? scratch_table : block_table;
    pg.dst_table = (j & 1) ? block_table : scratch_table;
    if (run_round_paged(plan[j], pg, src_has_deg, (int)LH, D, params->chunk, w, ws, stream) != cudaSuccess) return CKV_ERR_CUDA;
    src_has_deg = true;  // every round writes degrees
  }
  if (out_len) *out_len = plan.empty() ? len : plan.back().s_out;
  if (result_in_scratch) *result_in_scratch = (int32_t)(plan.size() & 1);
  return CKV_OK;
}

const char* ckv_status_string(int status) {
  switch (status) {
    case CKV_OK: return "ok";
    case CKV_ERR_INVALID_ARG: return "invalid argument";
    case CKV_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case CKV_ERR_CAPACITY: return "destination capacity too small";
    case CKV_ERR_WORKSPACE: return "workspace missing or too small";
    case CKV_ERR_NO_PROGRESS: return "ratio schedule merges nothing but the budget is not met";
    case CKV_ERR_UNSUPPORTED: return "unsupported shape or size";
    case CKV_ERR_CUDA: return "CUDA runtime error";
    default: return "unknown status";
  }
}

int ckv_compress_plan(int64_t len, const ckv_params* params, int64_t* out_len, int64_t* rounds,
                      int64_t* dst_cap) {
  int st = check_params(params);
  if (st != CKV_OK) return st;
  if (len < 0) return CKV_ERR_INVALID_ARG;
  std::vector<RoundPlan> plan;
  if ((st = plan_rounds(len, *params, plan)) != CKV_OK) return st;
  if (out_len) *out_len = plan.empty() ? len : plan.back().s_out;
  if (rounds) *rounds = (int64_t)plan.size();
  if (dst_cap) *dst_cap = dst_cap_needed(plan, len);
  return CKV_OK;
}

size_t ckv_workspace_bytes(const ckv_cache* shape, const ckv_params* params) {
  if (check_params(params) != CKV_OK || check_cache_shape(shape) != CKV_OK) return 0;
  const int64_t LH = (int64_t)shape->L * shape->H;
  const int es = esize_of(shape->dtype);
  std::vector<RoundPlan> plan;
  size_t need = 256;
  // prefill over the current length (an unreachable budget is reported by the call itself)
  if (plan_rounds(shape->len, *params, plan) == CKV_OK) {
    need = std::max(need, layout_workspace(LH, shape->D, es, params->chunk, plan, true).total);
  }
  // append: one window of `chunk` tokens, with a tmp window for odd round counts
  const ckv_params wp = window_params(*params);
  if (params->chunk > 0 && plan_rounds(params->chunk, wp, plan) == CKV_OK) {
    const size_t win = align_up((size_t)LH * params->chunk * shape->D * es) * 2 + align_up((size_t)LH * params->chunk * 4) * 2;
    need = std::max(need, layout_workspace(LH, shape->D, es, params->chunk, plan, false).total + win);
  }
  return need;
}

int ckv_compress_prefill(const ckv_cache* src, ckv_cache* dst, const ckv_params* params, int32_t* assign,
                         void* workspace, size_t workspace_bytes, void* cuda_stream, int64_t* rounds_done) {
  int st;
  if ((st = check_params(params)) != CKV_OK) return st;
  if ((st = check_cache_shape(src)) != CKV_OK) return st;
  if ((st = check_cache_shape(dst, false)) != CKV_OK) return st;
  if (src->L != dst->L || src->H != dst->H || src->D != dst->D || src->dtype != dst->dtype) return CKV_ERR_INVALID_ARG;
  if (!src->k || !src->v || !dst->k || !dst->v || !dst->deg) return CKV_ERR_INVALID_ARG;
  if (!aligned16(src->k) || !aligned16(src->v) || !aligned16(dst->k) || !aligned16(dst->v)) return CKV_ERR_ALIGNMENT;
  const int64_t LH = (int64_t)src->L * src->H;
  const int es = esize_of(src->dtype);
  const size_t src_bytes = (size_t)LH * src->cap * src->D * es, dst_bytes = (size_t)LH * dst->cap * dst->D * es;
  if (overlaps(src->k, src_bytes, dst->k, dst_bytes) || overlaps(src->v, src_bytes, dst->v, dst_bytes) ||
      overlaps(src->k, src_bytes, dst->v, dst_bytes) || overlaps(src->v, src_bytes, dst->k, dst_bytes))
    return CKV_ERR_INVALID_ARG;
  if (params->chunk == 0 && !bsm_supported(src->dtype, src->D)) return CKV_ERR_UNSUPPORTED;
  std::vector<RoundPlan> plan;
  if ((st = plan_rounds(src->len, *params, plan)) != CKV_OK) return st;
  if (dst->cap < dst_cap_needed(plan, src->len)) return CKV_ERR_CAPACITY;
  Workspace w = layout_workspace(LH, src->D, es, params->chunk, plan, assign != nullptr);
  const size_t need = w.total;
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return CKV_ERR_WORKSPACE;
  if (overlaps(workspace, need, dst->k, dst_bytes) || overlaps(workspace, need, dst->v, dst_bytes) ||
      overlaps(workspace, need, src->k, src_bytes) || overlaps(workspace, need, src->v, src_bytes))
    return CKV_ERR_INVALID_ARG;

  if (cudaMemsetAsync(workspace, 0, 256, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return CKV_ERR_CUDA;
  const Buf s{src->k, src->v, src->deg, src->logdeg, src->cap};
  const Buf d{dst->k, dst->v, dst->deg, dst->logdeg, dst->cap};
  st = run_plan(plan, s, d, src->len, (int)LH, src->D, src->dtype, params->chunk, assign, w,
                static_cast<unsigned char*>(workspace), static_cast<cudaStream_t>(cuda_stream));
  if (st != CKV_OK) return st;
  dst->len = plan.empty() ? src->len : plan.back().s_out;
  dst->pending = 0;
  if (rounds_done) *rounds_done = (int64_t)plan.size();
  return CKV_OK;
}

int ckv_compress_append(ckv_cache* cache, const void* k_new, const void* v_new, int32_t t_new,
                        const ckv_params* params, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int st;
  if ((st = check_params(params)) != CKV_OK) return st;
  if ((st = check_cache_shape(cache)) != CKV_OK) return st;
  if (t_new < 0 || (t_new > 0 && (!k_new || !v_new))) return CKV_ERR_INVALID_ARG;
  if (!cache->k || !cache->v || !cache->deg) return CKV_ERR_INVALID_ARG;
  if (!aligned16(cache->k) || !aligned16(cache->v) || !aligned16(k_new) || !aligned16(v_new)) return CKV_ERR_ALIGNMENT;
  if (params->chunk == 0) return CKV_ERR_INVALID_ARG;  // the append trigger is a window of `chunk` tokens
  if (cache->pending >= params->chunk) return CKV_ERR_INVALID_ARG;
  const int64_t LH = (int64_t)cache->L * cache->H;
  const int D = cache->D, es = esize_of(cache->dtype), c = params->chunk;
  const ckv_params wp = window_params(*params);
  std::vector<RoundPlan> plan;
  if ((st = plan_rounds(c, wp, plan)) != CKV_OK) return st;
  const int64_t win_out = plan.empty() ? c : plan.back().s_out;

  // host-side walk first: capacity must hold every intermediate state
  {
    int64_t len = cache->len, pend = cache->pending, peak = len;
    for (int32_t done = 0; done < t_new;) {
      const int32_t take = (int32_t)std::min<int64_t>(t_new - done, c - pend);
      len += take; pend += take; done += take;
      peak = std::max(peak, len);
      if (pend == c) { len -= c - win_out; pend = 0; }
    }
    if (peak > cache->cap) return CKV_ERR_CAPACITY;
  }
  Workspace w = layout_workspace(LH, D, es, c, plan, false);
  const size_t base = w.total;
  const size_t win_kv = align_up((size_t)LH * c * D * es), win_dg = align_up((size_t)LH * c * 4);
  if (!workspace || workspace_bytes < base + 2 * win_kv + 2 * win_dg || !aligned16(workspace)) return CKV_ERR_WORKSPACE;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  const Buf stage{ws + base, ws + base + win_kv, reinterpret_cast<int32_t*>(ws + base + 2 * win_kv),
                  reinterpret_cast<float*>(ws + base + 2 * win_kv + win_dg), c};
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, 256, stream) != cudaSuccess) return CKV_ERR_CUDA;

  for (int32_t done = 0; done < t_new;) {
    const int32_t take = (int32_t)std::min<int64_t>(t_new - done, c - cache->pending);
    CopyArgs cp{};  // K = [K, k], V = [V, v], N = [N, 1]
    cp.k_src = k_new; cp.v_src = v_new; cp.deg_src = nullptr;
    cp.k_dst = cache->k; cp.v_dst = cache->v; cp.deg_dst = cache->deg; cp.logdeg_dst = cache->logdeg;
    cp.src_cap = t_new; cp.dst_cap = cache->cap; cp.src_off = done; cp.dst_off = cache->len; cp.count = take;
    cp.LH = (int)LH;
    if (launch_copy(cp, cache->dtype, D, stream) != cudaSuccess) return CKV_ERR_CUDA;
    cache->len += take;
    cache->pending += take;
    done += take;
    if (cache->pending == c && !plan.empty()) {
      if ((st = cluster_window(cache, plan, win_out, LH, D, es, c, w, ws, stage, stream)) != CKV_OK) return st;
    }
    if (cache->pending == c) cache->pending = 0;
  }
  return CKV_OK;
}

int ckv_compress_append_batch(ckv_cache* caches, int32_t Bz, const void* k_new, const void* v_new, const ckv_params* params,
                              void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int st;
  if ((st = check_params(params)) != CKV_OK) return st;
  if (!caches || Bz <= 0 || !k_new || !v_new) return CKV_ERR_INVALID_ARG;
  if (params->chunk == 0) return CKV_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new)) return CKV_ERR_ALIGNMENT;
  const ckv_cache& c0 = caches[0];
  for (int32_t b = 0; b < Bz; ++b) {
    const ckv_cache& cb = caches[b];
    if ((st = check_cache_shape(&cb)) != CKV_OK) return st;
    if (cb.L != c0.L || cb.H != c0.H || cb.D != c0.D || cb.dtype != c0.dtype) return CKV_ERR_INVALID_ARG;
    if (!cb.k || !cb.v || !cb.deg) return CKV_ERR_INVALID_ARG;
    if (!aligned16(cb.k) || !aligned16(cb.v)) return CKV_ERR_ALIGNMENT;
    if (cb.pending >= params->chunk) return CKV_ERR_INVALID_ARG;
    if (cb.len + 1 > cb.cap) return CKV_ERR_CAPACITY;
  }
  const int64_t LH = (int64_t)c0.L * c0.H;
  const int D = c0.D, es = esize_of(c0.dtype), c = params->chunk;
  const ckv_params wp = window_params(*params);
  std::vector<RoundPlan> plan;
  if ((st = plan_rounds(c, wp, plan)) != CKV_OK) return st;
  const int64_t win_out = plan.empty() ? c : plan.back().s_out;
  Workspace w = layout_workspace(LH, D, es, c, plan, false);
  const size_t base = w.total;
  const size_t win_kv = align_up((size_t)LH * c * D * es), win_dg = align_up((size_t)LH * c * 4);
  if (!workspace || workspace_bytes < base + 2 * win_kv + 2 * win_dg || !aligned16(workspace)) return CKV_ERR_WORKSPACE;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  const Buf stage{ws + base, ws + base + win_kv, reinterpret_cast<int32_t*>(ws + base + 2 * win_kv),
                  reinterpret_cast<float*>(ws + base + 2 * win_kv + win_dg), c};
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, 256, stream) != cudaSuccess) return CKV_ERR_CUDA;

  // K = [K, k], V = [V, v], N = [N, 1] for every sequence: one launch per kAppendBatchMax sequences
  for (int32_t first = 0; first < Bz; first += kAppendBatchMax) {
    AppendBatchArgs a{};
    a.k_new = k_new; a.v_new = v_new;
    a.n = std::min<int32_t>(kAppendBatchMax, Bz - first);
    a.first = first; a.n_total = Bz; a.LH = (int32_t)LH;
    for (int32_t i = 0; i < a.n; ++i) {
      const ckv_cache& cb = caches[first + i];
      a.k[i] = cb.k; a.v[i] = cb.v; a.deg[i] = cb.deg; a.logdeg[i] = cb.logdeg;
      a.cap[i] = cb.cap; a.len[i] = cb.len;
    }
    if (launch_append_batch(a, c0.dtype, D, stream) != cudaSuccess) return CKV_ERR_CUDA;
  }
  for (int32_t b = 0; b < Bz; ++b) {
    ckv_cache* cb = &caches[b];
    cb->len += 1;
    cb->pending += 1;
    if (cb->pending == c) {
      if (!plan.empty() && (st = cluster_window(cb, plan, win_out, LH, D, es, c, w, ws, stage, stream)) != CKV_OK) return st;
      cb->pending = 0;
    }
  }
  return CKV_OK;
}

int ckv_compress_append_recluster(ckv_cache* cache, ckv_cache* spare, const void* k_new, const void* v_new, int32_t t_new,
                                  const ckv_params* params, int32_t interval, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream, int64_t* reclusterings) {
  int st;
  if ((st = check_params(params)) != CKV_OK) return st;
  if ((st = check_cache_shape(cache)) != CKV_OK) return st;
  if ((st = check_cache_shape(spare, false)) != CKV_OK) return st;
  if (params->budget <= 0 || interval <= 0) return CKV_ERR_INVALID_ARG;
  if (t_new < 0 || (t_new > 0 && (!k_new || !v_new))) return CKV_ERR_INVALID_ARG;
  if (cache->L != spare->L || cache->H != spare->H || cache->D != spare->D || cache->dtype != spare->dtype) return CKV_ERR_INVALID_ARG;
  if (!cache->k || !cache->v || !cache->deg || !spare->k || !spare->v || !spare->deg) return CKV_ERR_INVALID_ARG;
  if (!aligned16(cache->k) || !aligned16(cache->v) || !aligned16(spare->k) || !aligned16(spare->v) || !aligned16(k_new) ||
      !aligned16(v_new))
    return CKV_ERR_ALIGNMENT;
  const int64_t LH = (int64_t)cache->L * cache->H;
  const int D = cache->D, es = esize_of(cache->dtype);
  const int64_t trigger = params->budget + (int64_t)interval;
  if (cache->cap < trigger || spare->cap < trigger) return CKV_ERR_CAPACITY;
  const size_t a_bytes = (size_t)LH * cache->cap * D * es, b_bytes = (size_t)LH * spare->cap * D * es;
  if (overlaps(cache->k, a_bytes, spare->k, b_bytes) || overlaps(cache->v, a_bytes, spare->v, b_bytes) ||
      overlaps(cache->k, a_bytes, spare->v, b_bytes) || overlaps(cache->v, a_bytes, spare->k, b_bytes))
    return CKV_ERR_INVALID_ARG;
  ckv_params one = *params;  // Algorithm 1 calls CentroidKV once per trigger
  one.n_rounds_max = 1;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);

  // The lengths are a function of shapes only: walk the steps on the host first, so that an unreachable budget or
  // a short workspace is reported before anything is enqueued; then walk them again and launch.
  for (int pass = 0; pass < 2; ++pass) {
    const bool dry = pass == 0;
    ckv_cache live = *cache, other = *spare;
    int64_t calls = 0;
    // the status word is defined after every call, also one that only appends
    if (!dry && workspace && workspace_bytes >= 256 && cudaMemsetAsync(workspace, 0, 256, stream) != cudaSuccess) return CKV_ERR_CUDA;
    for (int32_t done = 0; done < t_new || live.len >= trigger;) {
      if (live.len >= trigger) {
        // `if s >= B + g`: one round over the whole cache into the other buffer, then the buffers trade places
        std::vector<RoundPlan> plan;
        if ((st = plan_rounds(live.len, one, plan)) != CKV_OK) return st;
        if (plan.empty() || plan.back().s_out >= live.len) return CKV_ERR_NO_PROGRESS;
        Workspace w = layout_workspace(LH, D, es, one.chunk, plan, false);
        if (dry) {
          if (!workspace || workspace_bytes < w.total || !aligned16(workspace)) return CKV_ERR_WORKSPACE;
        } else {
          const Buf src{live.k, live.v, live.deg, live.logdeg, live.cap};
          const Buf dst{other.k, other.v, other.deg, other.logdeg, other.cap};
          if ((st = run_plan(plan, src, dst, live.len, (int)LH, D, live.dtype, one.chunk, nullptr, w, ws, stream)) != CKV_OK) return st;
        }
        std::swap(live.k, other.k);
        std::swap(live.v, other.v);
        std::swap(live.deg, other.deg);
        std::swap(live.logdeg, other.logdeg);
        std::swap(live.cap, other.cap);
        live.len = plan.back().s_out;
        ++calls;
        continue;
      }
      const int32_t take = (int32_t)std::min<int64_t>(t_new - done, trigger - live.len);
      if (!dry) {
        CopyArgs cp{};  // K = [K, k], V = [V, v], N = [N, 1]
        cp.k_src = k_new; cp.v_src = v_new; cp.deg_src = nullptr;
        cp.k_dst = live.k; cp.v_dst = live.v; cp.deg_dst = live.deg; cp.logdeg_dst = live.logdeg;
        cp.src_cap = t_new; cp.dst_cap = live.cap; cp.src_off = done; cp.dst_off = live.len; cp.count = take;
        cp.LH = (int)LH;
        if (launch_copy(cp, live.dtype, D, stream) != cudaSuccess) return CKV_ERR_CUDA;
      }
      live.len += take;
      done += take;
    }
    if (!dry) {
      live.pending = 0;
      other.len = 0;
      other.pending = 0;
      *cache = live;
      *spare = other;
      if (reclusterings) *reclusterings = calls;
    }
  }
  return CKV_OK;
}

int ckv_workspace_status(const void* workspace, void* cuda_stream, int32_t* status_host) {
  if (!workspace || !status_host) return CKV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(status_host, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return CKV_ERR_CUDA;
  return cudaStreamSynchronize(st) == cudaSuccess ? CKV_OK : CKV_ERR_CUDA;
}

size_t ckv_decode_workspace_bytes(int32_t Bz, int32_t H, int32_t G, int32_t D, int64_t max_len) {
  if (Bz <= 0 || H <= 0 || G <= 0 || D <= 0 || max_len < 0) return 0;
  return align_up(decode_partial_floats(Bz, H, G, D, max_len) * sizeof(float)) + 256;
}

int ckv_decode_attn(const ckv_layer_view* views_dev, int32_t Bz, int32_t H, int32_t G, int32_t D, int32_t dtype,
                    const void* q, void* out, float scale, int64_t max_len, void* workspace, size_t workspace_bytes,
                    void* cuda_stream) {
  if (!views_dev || !q || !out || Bz <= 0 || H <= 0 || G <= 0 || max_len < 0) return CKV_ERR_INVALID_ARG;
  if (dtype != CKV_F32 && dtype != CKV_BF16) return CKV_ERR_INVALID_ARG;
  if (D != 128 || G > 8 || H > 65535 || Bz > 65535) return CKV_ERR_UNSUPPORTED;
  if (!aligned16(q) || !aligned16(out)) return CKV_ERR_ALIGNMENT;
  const size_t need = ckv_decode_workspace_bytes(Bz, H, G, D, max_len);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return CKV_ERR_WORKSPACE;
  DecodeArgs a{};
  a.views = views_dev; a.q = q; a.out = out;
  a.partial = static_cast<float*>(workspace);
  a.Bz = Bz; a.H = H; a.G = G;
  decode_plan(Bz, H, dtype, max_len, 0, G, D, &a.n_splits, &a.span);
  a.max_len = max_len;
  a.scale = scale;
  return launch_decode(a, dtype, D, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? CKV_OK : CKV_ERR_CUDA;
}

}  // extern "C"
